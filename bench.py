#!/usr/bin/env python
"""Benchmark of the SwitchHead layer forward pass (one step = one sh_forward over one batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

Prints ONE JSON line.  `value` = tokens/s with x already resident in HBM, L2 flushed before
every timed step; `e2e` = the same metric with x in pinned host memory and the result copied
back inside the timed region; `roofline` = the kernel with the longest span INSIDE the real
pass (device-clock stamps of sh_forward_stamped: same launches as sh_forward) against the
measured bf16 tensor peak (MEASURED_PEAKS.json); `per_config` = the same figures for every
bf16 workload; `cpu_baseline` = the fp64 oracle on the host cores.

With --gpus N > 1 and no torchrun environment the script starts its own N ranks (torch.distributed.run,
rendezvous on 127.0.0.1).  Every rank runs the same workload on its own batch (independent
sequences, no collective on the data path); a barrier brackets the timed region and the slowest
rank sets the time.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

DEFAULT_CONFIG = "c4_262m_bf16"
BF16_CONFIGS = ["small_bf16", "c4_262m_bf16", "long_ctx_bf16", "wide_skew_bf16"]
# dram__bytes_read.sum + dram__bytes_write.sum per launch of each kernel (MB), from the one-kernel ncu
# captures summarised under profiles/ (the file named beside each workload)
DRAM_TRAFFIC_MB = {
    # ("qk" and "gate": where the one-grid front serves the workload - all but wide_skew_bf16 - they are ONE kernel
    #  that reads x once: its figure stands under both names)
    "c4_262m_bf16": {"gate": 19.02, "qk": 19.02, "v": 21.66, "attn": 25.23, "o": 13.17},        # profiles/c4_262m_bf16_forward_kernels.md
    "long_ctx_bf16": {"gate": 38.60, "qk": 38.60, "v": 43.71, "attn": 52.79, "o": 38.10},        # profiles/long_ctx_bf16_forward_kernels.md
    "small_bf16": {"gate": 8.76, "qk": 8.76, "v": 11.84, "attn": 6.34, "o": 3.18},               # profiles/small_bf16_forward_kernels.md
    "wide_skew_bf16": {"gate": 84.90, "sort": 4.39, "qk": 109.21, "v": 600.48, "attn": 143.04, "o": 618.35},   # profiles/wide_skew_bf16_forward_kernels.md
}
KERNEL_STAGE = {"gate": "gate_topk_sort", "sort": "gate_topk_sort", "qk_a": "qk_proj", "qk_b": "qk_proj", "v": "v_experts",
                "attn": "attention", "o": "o_experts"}
STAGES = ["gate_topk_sort", "qk_proj", "v_experts", "attention", "o_experts"]
METRIC = "switchhead_layer_fwd_tokens_per_s"
MIN_TIMED_SECONDS = 0.5        # the timed region is repeated until it has run this long (clock samples need load to see)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(tflops=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"],
                    hbm_gbs=p["hbm_gbs"], source="measured")
    return dict(tflops=1590.0, tflops_sustained=1400.0, hbm_gbs=6650.0, source="fallback")


def config_dict(cfg, world, args):
    """The workload description both arms print (identical keys and values)."""
    return {"workload": cfg.name, "batch_per_gpu": cfg.batch, "seq_len": cfg.seq, "d_model": cfg.d_model,
            "n_heads": cfg.n_heads, "d_head": cfg.d_head, "n_experts": cfg.n_experts, "k": cfg.k,
            "causal": True, "rope_base": args.rope if args.rope > 0 else None,
            "shared_selection": bool(args.shared_selection),
            "l2": "flushed before every timed step (256 MiB write)",
            "parallelism": f"batch-sharded replicas x{world}, no collective"}


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}",
                                       "--format=csv,noheader,nounits", "-lms", "5"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        rows = [l.strip().split(", ") for l in self.f if l.strip()]
        self.f.close()
        os.unlink(self.f.name)
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.strip().lower().startswith("active"):
                    reasons.add(n)
        if sm:
            # samples under load: those drawing more than the midpoint between idle and peak power
            thr = 0.5 * (min(pw) + max(pw))
            hot = [s for s, p in zip(sm, pw) if p >= thr] or sm
            out.update(sm_mhz=float(np.median(hot)), sm_max_mhz=float(max(mx)), samples=len(sm), samples_under_load=len(hot),
                       power_w_max=float(max(pw)))
        out["reasons"] = sorted(reasons)
        return out


def oracle_sample(cfg, inp, seconds_budget=12.0, rope_base=None, shared_selection=False):
    """Times the oracle, as it stands, on whole sequences of the workload (batch elements are
    independent), cycling through the batch until about `seconds_budget` seconds are spent."""
    from oracle.switchhead_oracle import switchhead_forward
    B = inp.x.shape[0]
    done, t_used = 0, 0.0
    t0 = time.perf_counter()
    nb = 1
    while True:
        lo = done % B
        nb = min(nb, B - lo)
        t1 = time.perf_counter()
        switchhead_forward(inp.x[lo:lo + nb], inp.Wq, inp.Wk, inp.Wv, inp.Wo, inp.Ws, inp.Wd, cfg.k,
                           inp.bias_s, inp.bias_d, return_stages=False, rope_base=rope_base,
                           shared_selection=shared_selection)
        dt = time.perf_counter() - t1
        done += nb
        t_used = time.perf_counter() - t0
        if t_used + 2 * dt > seconds_budget:
            break
        nb = min(2 * nb, B)
    tokens = done * inp.x.shape[1]
    return tokens / t_used, done, t_used


def run_reference(args, rank, world):
    """--impl reference: the fp64 oracle, as it stands, on the host cores (rank 0 only)."""
    if rank != 0:
        return
    from paper_2312_07987_b200 import inputs
    cfg = inputs.CONFIGS[args.config]
    # a bounded sample per step: a few whole sequences of the workload
    sample_b = max(1, min(cfg.batch, 2 if cfg.seq <= 1024 else 1))
    inp = inputs.make_inputs(cfg, batch=sample_b)
    from oracle.switchhead_oracle import switchhead_forward
    run = lambda: switchhead_forward(inp.x, inp.Wq, inp.Wk, inp.Wv, inp.Wo, inp.Ws, inp.Wd, cfg.k,
                                     inp.bias_s, inp.bias_d, return_stages=False,
                                     rope_base=args.rope if args.rope > 0 else None,
                                     shared_selection=args.shared_selection)
    for _ in range(min(args.warmup, 1)):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    dt = time.perf_counter() - t0
    tokens = sample_b * cfg.seq
    value = tokens * args.steps / dt
    cores = len(os.sched_getaffinity(0))
    sample = f"{sample_b} of {cfg.batch} sequences of {cfg.seq} tokens per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg, world, args),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def launch_ranks(n: int) -> int:
    """--gpus N without a torchrun environment: start N ranks of this script on this node."""
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def timed_region(layer, x, out, flush, stream, steps, barrier, min_seconds, lead_in=3):
    """Runs the K-step timed region (flush, event, sh_forward, event) again and again until it has been
    running for min_seconds; returns the per-repeat mean milliseconds per step.  Every repeat starts,
    behind its barrier, with `lead_in` untimed steps: a pass is ten launches, and until the host is a few
    launches ahead of the device the gaps between them sit inside the first steps' event pairs (with
    K = 50 the mean read 116 us against 103 us with K = 200)."""
    import torch
    means = []
    t_begin = time.perf_counter()
    while True:
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for _ in range(lead_in):
            flush.fill_(1)
            layer.sh_forward(x, out)
        for a, b in ev:
            flush.fill_(1)
            a.record(stream)
            layer.sh_forward(x, out)
            b.record(stream)
        barrier()
        means.append(float(np.mean([a.elapsed_time(b) for a, b in ev])))
        if (time.perf_counter() - t_begin >= min_seconds and len(means) >= 3) or len(means) >= 400:   # (>= 3: one stalled repeat must not be the result)
            return means


def kernel_timeline(layer, x, out, flush, reps=12):
    """Mean per-kernel spans inside the real pass, microseconds from the pass's first stamp:
    {kernel: (start, end)} (start = first CTA past its dependency wait, end = last CTA done)."""
    import torch
    acc = {}
    for _ in range(reps):
        flush.fill_(1)
        torch.cuda.synchronize()
        st = layer.sh_forward_stamped(x, out)
        t0 = min(v[0] for v in st.values())
        for k, (res, start, end) in st.items():
            a = acc.setdefault(k, [0.0, 0.0, 0])
            a[0] += (start - t0) * 1e-3; a[1] += (end - t0) * 1e-3; a[2] += 1
    return {k: (a[0] / a[2], a[1] / a[2]) for k, a in acc.items()}


def roofline_from_timeline(cfg, tl, fl, peaks):
    """The kernel with the longest span inside the pass, against the bound that applies to it."""
    N = cfg.n_tokens
    span = {k: e - s for k, (s, e) in tl.items()}
    if "qk_a" in span and "qk_b" in span:           # two grids of one projection: one span
        s0 = min(tl["qk_a"][0], tl["qk_b"][0]); e0 = max(tl["qk_a"][1], tl["qk_b"][1])
        span["qk_a"] = e0 - s0
        del span["qk_b"]
    dom = max(span, key=span.get)
    us = span[dom]
    flop = {"qk_a": fl["qk"], "v": fl["v"], "attn": fl["attn_half"], "o": fl["o"]}
    traffic = DRAM_TRAFFIC_MB.get(cfg.name, {}).get(dom.replace("_a", ""))
    if dom in ("gate", "sort"):
        bytes_ = N * cfg.d_model * 2 + 4 * (2 * N * cfg.n_heads * cfg.k) * 4        # x read once + idx/gate/lists written
        ach = bytes_ / (us * 1e-6) / 1e9
        roof = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"])
    else:
        ach = flop[dom] / (us * 1e-6) / 1e12
        roof = dict(bound="tensor", achieved=ach, peak=peaks["tflops"], unit="TFLOP/s", frac=ach / peaks["tflops"])
    roof.update(kernel=KERNEL_STAGE[dom], ms=us * 1e-3, peak_source=peaks["source"],
                timing="span of the kernel inside the real pass (device-clock stamps, first CTA past its dependency wait to last CTA done)",
                traffic=None if traffic is None else traffic * 1e6, traffic_unit="bytes per launch (ncu)")
    if dom == "o":
        # the on-chip sum multiplies every token tile by all E experts of a head (zero rows for the
        # tokens that did not select one): logical tensor work = E/k times the useful work counted here;
        # where the selection is 2:4 sparse along the expert-innermost contraction axis (k <= 2, E = 4
        # or 8, d_head 128, <= 4 heads) the sparse instruction does that product in half the cycles
        sparse = cfg.k <= 2 and cfg.n_experts in (4, 8) and 64 < cfg.d_head <= 128 and cfg.n_heads <= 4
        roof["executed_over_useful_flop"] = cfg.n_experts / cfg.k
        roof["tensor_cycles_over_useful"] = cfg.n_experts / cfg.k / (2 if sparse else 1)
        roof["o_kernel"] = "2:4-sparse CTA-pair kernel" if sparse else "masked kernel"
    return roof


def measure_config(cfg, args, rank, world, peaks, flush, barrier, steps, min_seconds, with_e2e):
    """Everything measured for one workload on this rank; the caller takes the max over ranks."""
    import torch
    from paper_2312_07987_b200 import binding, inputs, sharding
    inp = inputs.make_inputs(cfg)
    inp.x = sharding.rank_batch(inp.x, rank)                                 # rows keep their gate margins
    layer = binding.layer_from_inputs(inp, shared_selection=args.shared_selection)
    if args.rope > 0:
        layer.sh_set_rope(args.rope)
    x = binding.to_device(inp.x, cfg.dtype)
    out = torch.empty(inp.x.shape, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        layer.sh_forward(x, out)
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0, "device status word set during warm-up"
    res = dict(launches=layer.sh_launch_count())

    res["repeat_means"] = timed_region(layer, x, out, flush, stream, steps, barrier, min_seconds)

    # L2-warm variant: K back-to-back calls, one event pair
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    for _ in range(3):                                      # (untimed lead-in, as in timed_region)
        layer.sh_forward(x, out)
    a.record(stream)
    for _ in range(steps):
        layer.sh_forward(x, out)
    b.record(stream)
    torch.cuda.synchronize()
    res["warm_ms"] = a.elapsed_time(b) / steps
    # the same with the pass captured once in a CUDA graph and replayed (the caller's option: the library's
    # launches, side streams included, are capturable): one host call per pass instead of ~15, so the
    # figure is the device's back-to-back time even where the host cannot keep ahead
    res["graph_ms"] = None
    try:
        gstream = torch.cuda.Stream()
        with torch.cuda.stream(gstream):
            layer.sh_forward(x, out)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=gstream):
                layer.sh_forward(x, out)
            for _ in range(3):
                graph.replay()
            a.record(gstream)
            for _ in range(steps):
                graph.replay()
            b.record(gstream)
        torch.cuda.synchronize()
        res["graph_ms"] = a.elapsed_time(b) / steps
        del graph
    except Exception as e:                                   # (reported as null; the launch path does not depend on it)
        res["graph_error"] = str(e)[:200]
        torch.cuda.synchronize()

    res["timeline"] = kernel_timeline(layer, x, out, flush)
    # serialised stage times (ordinary launches, one stream, CUDA events at the stage boundaries): what each
    # stage costs ALONE; they add up to more than a pass, in which the kernels overlap
    # (two untimed calls first: a stage-timed pass launches the front's three kernels one by one, which an
    #  ordinary pass of this workload never does - their first launches set function attributes on the host)
    for _ in range(2):
        layer.sh_forward_timed(x, out)
    stage = np.zeros(6)
    for _ in range(6):
        flush.fill_(1)
        stage += np.array(layer.sh_forward_timed(x, out))
    res["stage_ms_serialised"] = stage / 6

    if with_e2e:
        # end to end with host buffers: every step copies x in from pinned host memory and the result back
        # out; the three run as a pipeline on three streams (pipeline.HostFedLayer), as a host-fed caller would
        from paper_2312_07987_b200 import pipeline
        xh = [x.cpu().pin_memory() for _ in range(2)]
        outh = [torch.empty(inp.x.shape, dtype=torch.float32).pin_memory() for _ in range(2)]
        pipe = pipeline.HostFedLayer(layer, x)
        for i in range(4):
            pipe.step(xh[i & 1], outh[i & 1])
        pipe.wait()
        ref = out.cpu()
        assert torch.equal(outh[1], ref) or float((outh[1] - ref).abs().max()) < 1e-2 * float(ref.abs().max()), \
            "pipelined result differs from the direct one"
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(pipe.s_in)
        for i in range(steps):
            pipe.step(xh[i & 1], outh[i & 1])
        b.record(pipe.s_out)
        pipe.wait()
        barrier()
        res["e2e_ms_f32_result"] = a.elapsed_time(b)
        res["h2d"] = int(x.numel() * x.element_size())
        res["d2h_f32_result"] = int(out.numel() * 4)
        # the same with the result rounded to fp16 on its way out of the output projection (sh_set_output_f16):
        # half the bytes on the way back, which is what bounds a host-fed step
        layer.sh_set_output_f16(True)
        outh16 = [torch.empty(inp.x.shape, dtype=torch.float16).pin_memory() for _ in range(2)]
        pipe16 = pipeline.HostFedLayer(layer, x)
        for i in range(4):
            pipe16.step(xh[i & 1], outh16[i & 1])
        pipe16.wait()
        r16 = ref.to(torch.float16)
        assert torch.equal(outh16[1], r16) or float((outh16[1].float() - ref).abs().max()) < 1e-2 * float(ref.abs().max()), \
            "pipelined fp16 result differs from the direct one"
        barrier()
        a.record(pipe16.s_in)
        for i in range(steps):
            pipe16.step(xh[i & 1], outh16[i & 1])
        b.record(pipe16.s_out)
        pipe16.wait()
        barrier()
        res["e2e_ms"] = a.elapsed_time(b)
        res["d2h"] = int(out.numel() * 2)
        layer.sh_set_output_f16(False)
    assert layer.sh_last_status() == 0, "device status word set during the timed region"
    res["inp"], res["x"], res["out"] = inp, x, out
    layer.close()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default=DEFAULT_CONFIG)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the table over the other workloads")
    ap.add_argument("--shared-selection", action="store_true",
                    help="one gate for the source and the destination side (the paper's Shared Selection variant)")
    ap.add_argument("--rope", type=float, default=0.0,
                    help="rotary position embeddings on Q, K with this base (0 = off, the headline configuration)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(launch_ranks(args.gpus))                 # this process becomes the launcher of N ranks

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2312_07987_b200 import binding, inputs, sharding

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    cfg = inputs.CONFIGS[args.config]
    peaks = load_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")       # > 126 MB L2

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    m = measure_config(cfg, args, rank, world, peaks, flush, barrier, args.steps, MIN_TIMED_SECONDS, with_e2e=True)
    clocks = sampler.stop() if sampler else None

    # ---- max over ranks (every repeat mean, so that the median is of the slowest rank's times) ----
    nrep = int(sharding.max_over_ranks([-float(len(m["repeat_means"]))], device="cuda")[0] * -1)   # fewest repeats any rank made
    reduced = sharding.max_over_ranks(m["repeat_means"][:nrep] + [m["e2e_ms"], m["warm_ms"], m["e2e_ms_f32_result"]], device="cuda")
    repeat_means, e2e_ms, warm_ms, e2e_ms_f32 = reduced[:nrep], reduced[nrep], reduced[nrep + 1], reduced[nrep + 2]

    line = None
    if rank == 0:
        N = cfg.n_tokens
        fl = inputs.useful_flop(cfg)
        ms_step = float(np.median(repeat_means))
        value = sharding.aggregate_throughput(N, world, ms_step * 1e-3)
        useful_tflops = world * fl["total"] / (ms_step * 1e-3) / 1e12
        tl = m["timeline"]
        line = {
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == inputs.DTYPE_BF16 else "f32",
            "data": "synthetic",
            "config": config_dict(cfg, world, args),
            "timed_region": {"repeats": len(repeat_means), "steps_per_repeat": args.steps, "untimed_lead_in_steps_per_repeat": 3,
                             "ms_per_step": "median over the repeats of the mean over a repeat's steps",
                             "repeat_min_ms": float(min(repeat_means)), "repeat_max_ms": float(max(repeat_means))},
            "useful_tflops": useful_tflops,
            "frac_of_bf16_peak_measured": useful_tflops / (world * peaks["tflops"]),
            "frac_of_bf16_peak_nominal_2250": useful_tflops / (world * 2250.0),
            "ms_per_step_l2_warm": warm_ms,
            "ms_per_step_l2_warm_graph_replay": m.get("graph_ms"),
            "useful_tflops_l2_warm": world * fl["total"] / (warm_ms * 1e-3) / 1e12,
            "kernel_spans_us": {k: [round(s, 2), round(e, 2)] for k, (s, e) in sorted(tl.items(), key=lambda kv: kv[1][0])},
            "stage_ms_serialised": {n: float(v) for n, v in zip(STAGES + ["total"], m["stage_ms_serialised"])},
            "gpu_launches": m["launches"] * args.steps * len(repeat_means),
            "launches_per_step": m["launches"],
            "e2e": {"value": world * N * args.steps / (e2e_ms * 1e-3), "unit": "tokens/s",
                    "h2d_bytes_per_step": m["h2d"], "d2h_bytes_per_step": m["d2h"],
                    "result_dtype": "f16 (sh_set_output_f16: the fp32 result rounded once by the output projection's epilogue)",
                    "with_f32_result": {"value": world * N * args.steps / (e2e_ms_f32 * 1e-3), "unit": "tokens/s",
                                        "d2h_bytes_per_step": m["d2h_f32_result"]}},
            "roofline": roofline_from_timeline(cfg, tl, fl, peaks),
            "clocks": clocks,
        }
        # ---- dense multi-head comparator on the same x (262M-scale workload only) ----
        if cfg.name == "c4_262m_bf16" and not args.no_dense:
            x, out = m["x"], m["out"]
            stream = torch.cuda.current_stream()
            Wq, Wk, Wv, Wo = inputs.make_dense_mha_weights(cfg.d_model, 16, 64, seed=102, dtype=cfg.dtype)
            dl = binding.Layer(cfg.d_model, 16, 64, dense=True)
            dl.sh_configure(cfg.dtype, cfg.batch, cfg.seq)
            dv = lambda t: binding.to_device(t, cfg.dtype)
            dl.sh_set_weights(dv(Wq), dv(Wk), dv(Wv[:, None]), dv(Wo[:, None]))
            for _ in range(3):
                dl.sh_forward(x, out)
            torch.cuda.synchronize()
            dt = []
            for _ in range(50):
                flush.fill_(1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream); dl.sh_forward(x, out); b.record(stream)
                torch.cuda.synchronize()
                dt.append(a.elapsed_time(b))
            dms = float(np.median(dt))
            dense_flop = 2.0 * N * cfg.d_model * 3 * 1024 + 2.0 * cfg.batch * 16 * cfg.seq ** 2 * 64 + 2.0 * N * 1024 * cfg.d_model
            line["dense_mha_16x64"] = {"ms_per_step": dms, "switchhead_over_dense_time": ms_step / dms,
                                       "useful_tflops": dense_flop / (dms * 1e-3) / 1e12,
                                       "note": "same attention kernel (exp-bound at d_head 64); its fused Q/K/V projection and its output "
                                               "projection both on the CTA-pair GEMM kernel (256 x 256 tiles)"}
            dl.close()
        # ---- the same layer as the paper's main models run it: with a Transformer-XL cache of one chunk (C = 2) ----
        if cfg.name == "c4_262m_bf16" and not args.no_dense:
            import dataclasses
            cx = dataclasses.replace(cfg, name="c4_262m_bf16+cache", seq=2 * cfg.seq)
            ix = inputs.make_inputs(cx, enforce_gap=False)
            lx = binding.layer_from_inputs(ix, cache_len=cfg.seq)
            # relative positions as in Transformer-XL: random projection and bias vectors of the trained model's shapes
            rg = np.random.Generator(np.random.PCG64(103))
            Wr = torch.from_numpy((rg.standard_normal((cfg.n_heads, cfg.d_model, cfg.d_head)) / np.sqrt(cfg.d_model)).astype(np.float32)).cuda()
            uu = torch.from_numpy((0.5 * rg.standard_normal((cfg.n_heads, cfg.d_head))).astype(np.float32)).cuda()
            vv = torch.from_numpy((0.5 * rg.standard_normal((cfg.n_heads, cfg.d_head))).astype(np.float32)).cuda()
            xx = binding.to_device(ix.x, cfg.dtype)
            ox = torch.empty((cfg.batch, cfg.seq, cfg.d_model), dtype=torch.float32, device="cuda")
            stream = torch.cuda.current_stream()
            for _ in range(3):
                lx.sh_forward(xx, ox)
            torch.cuda.synchronize()
            dt = []
            for _ in range(50):
                flush.fill_(1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream); lx.sh_forward(xx, ox); b.record(stream)
                torch.cuda.synchronize()
                dt.append(a.elapsed_time(b))
            assert lx.sh_last_status() == 0
            Tc = cfg.seq
            # keys and values (k experts) over cache + chunk, Q and O over the chunk; a query sees Tc + (t + 1) keys
            fx = (2.0 * (2 * N) * cfg.d_model * cfg.n_heads * cfg.d_head + 2.0 * N * cfg.d_model * cfg.n_heads * cfg.d_head
                  + 2.0 * (2 * N) * cfg.n_heads * cfg.k * cfg.d_model * cfg.d_head + 2.0 * N * cfg.n_heads * cfg.k * cfg.d_head * cfg.d_model
                  + 4.0 * cfg.batch * cfg.n_heads * cfg.d_head * (cfg.seq * Tc + cfg.seq * cfg.seq / 2))
            xms = float(np.median(dt))
            lx.sh_set_xl_positions(Wr, uu, vv)
            for _ in range(3):
                lx.sh_forward(xx, ox)
            torch.cuda.synchronize()
            dtp = []
            for _ in range(50):
                flush.fill_(1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream); lx.sh_forward(xx, ox); b.record(stream)
                torch.cuda.synchronize()
                dtp.append(a.elapsed_time(b))
            assert lx.sh_last_status() == 0
            pms = float(np.median(dtp))
            # position term: the score-bias GEMM Q R^T over the visible distances (causal part counted as for attention)
            fpos = 2.0 * cfg.batch * cfg.n_heads * cfg.d_head * (cfg.seq * Tc + cfg.seq * cfg.seq / 2)
            line["xl_context_c2"] = {"cache_len": Tc, "chunk_tokens_per_step": N, "ms_per_step": xms,
                                     "chunk_tokens_per_s": N / (xms * 1e-3), "useful_tflops": fx / (xms * 1e-3) / 1e12,
                                     "with_relative_positions": {"ms_per_step": pms, "chunk_tokens_per_s": N / (pms * 1e-3),
                                                                 "useful_tflops": (fx + fpos) / (pms * 1e-3) / 1e12},
                                     "note": "x = [cache; chunk] per sequence, out for the chunk; first figure: scores q.k; "
                                             "second: with Transformer-XL's relative-position term (the paper's main configuration)"}
            lx.close()
        if not args.no_cpu_baseline:
            v, nseq, secs = oracle_sample(cfg, m["inp"], rope_base=args.rope if args.rope > 0 else None,
                                          shared_selection=args.shared_selection)
            line["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": len(os.sched_getaffinity(0)),
                                    "kind": "oracle",
                                    "sample": f"{nseq} sequences of {cfg.seq} tokens drawn from the workload's {cfg.batch}, {secs:.1f} s, fp64 numpy"}
        line["paper_context"] = "paper reports 44% of dense MACs and 27% of dense activation memory at 262M params (analytic); no layer timing"
    del m

    # ---- the other bf16 workloads (a few milliseconds of GPU time each): one record per config ----
    if not args.no_per_config:
        per = {}
        for name in BF16_CONFIGS:
            c = inputs.CONFIGS[name]
            if name == cfg.name:
                if rank == 0:
                    per[name] = dict(ms_per_step=line["ms_per_step"], useful_tflops=line["useful_tflops"] / world,
                                     frac_of_bf16_peak_measured=line["frac_of_bf16_peak_measured"],
                                     ms_per_step_l2_warm=line["ms_per_step_l2_warm"],
                                     ms_per_step_l2_warm_graph_replay=line["ms_per_step_l2_warm_graph_replay"],
                                     dominant_kernel=line["roofline"]["kernel"], dominant_kernel_ms=line["roofline"]["ms"],
                                     dominant_kernel_frac=line["roofline"]["frac"])
                continue
            steps_c = 50 if c.n_tokens * c.d_model < (1 << 25) else 20
            mc = measure_config(c, args, rank, world, peaks, flush, barrier, steps_c, 0.1, with_e2e=False)
            nrep = int(sharding.max_over_ranks([-float(len(mc["repeat_means"]))], device="cuda")[0] * -1)
            red = sharding.max_over_ranks(mc["repeat_means"][:nrep] + [mc["warm_ms"]], device="cuda")
            if rank == 0:
                flc = inputs.useful_flop(c)
                msc = float(np.median(red[:nrep]))
                roof = roofline_from_timeline(c, mc["timeline"], flc, peaks)
                per[name] = dict(ms_per_step=msc, useful_tflops=flc["total"] / (msc * 1e-3) / 1e12,
                                 frac_of_bf16_peak_measured=flc["total"] / (msc * 1e-3) / 1e12 / peaks["tflops"],
                                 ms_per_step_l2_warm=red[nrep], ms_per_step_l2_warm_graph_replay=mc.get("graph_ms"),
                                 dominant_kernel=roof["kernel"], dominant_kernel_ms=roof["ms"],
                                 dominant_kernel_frac=roof["frac"],
                                 kernel_spans_us={k: [round(s, 2), round(e, 2)] for k, (s, e) in sorted(mc["timeline"].items(), key=lambda kv: kv[1][0])})
            del mc
        if rank == 0:
            line["per_config"] = per

    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
