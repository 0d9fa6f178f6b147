#!/usr/bin/env python
"""Benchmark of the SwitchHead layer forward pass (one step = one sh_forward over one batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

Prints ONE JSON line.  `value` = tokens/s with x already resident in HBM (L2 flushed
between timed steps); `e2e` = the same metric with x in pinned host memory and the result
copied back inside the timed region; `roofline` = the dominant stage against the measured
bf16 tensor peak (MEASURED_PEAKS.json); `cpu_baseline` = the fp64 oracle on the host cores.
With N > 1 (torchrun) every rank runs the same workload on its own batch (independent
sequences, no collective on the data path) and the slowest rank sets the time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

DEFAULT_CONFIG = "c4_262m_bf16"
# dram__bytes_read.sum + dram__bytes_write.sum per launch of each stage's main kernel, from the ncu
# capture summarised in profiles/c4_262m_bf16_forward_kernels.md (MB, workload c4_262m_bf16)
DRAM_TRAFFIC_MB = {"c4_262m_bf16": {"gate_topk_sort": 16.92, "qk_proj": 18.91, "v_experts": 29.92,
                                    "attention": 25.22, "o_experts": 13.23}}
STAGES = ["gate_topk_sort", "qk_proj", "v_experts", "attention", "o_experts"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(tflops=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"],
                    hbm_gbs=p["hbm_gbs"], source="measured")
    return dict(tflops=1590.0, tflops_sustained=1400.0, hbm_gbs=6650.0, source="fallback")


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}",
                                       "--format=csv,noheader,nounits", "-lms", "20"],
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
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.strip().lower().startswith("active"):
                    reasons.add(n)
        if sm:
            hot = sorted(sm)[len(sm) // 2:]            # upper half = samples under load
            out.update(sm_mhz=float(np.median(hot)), sm_max_mhz=float(max(mx)), samples=len(sm))
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
        "impl": "reference", "metric": "switchhead_layer_fwd_tokens_per_s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": cfg.batch, "seq_len": cfg.seq, "d_model": cfg.d_model,
                   "n_heads": cfg.n_heads, "d_head": cfg.d_head, "n_experts": cfg.n_experts, "k": cfg.k},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default=DEFAULT_CONFIG)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--shared-selection", action="store_true",
                    help="one gate for the source and the destination side (the paper's Shared Selection variant)")
    ap.add_argument("--rope", type=float, default=0.0,
                    help="rotary position embeddings on Q, K with this base (0 = off, the headline configuration)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

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

    # each rank owns its own batch of independent sequences (same weights, rank-specific x)
    inp = inputs.make_inputs(cfg)
    inp.x = sharding.rank_batch(inp.x, rank)                                 # rows keep their gate margins
    layer = binding.layer_from_inputs(inp, shared_selection=args.shared_selection)
    if args.rope > 0:
        layer.sh_set_rope(args.rope)
    x = binding.to_device(inp.x, cfg.dtype)
    out = torch.empty(inp.x.shape, dtype=torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")       # > 126 MB L2
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        layer.sh_forward(x, out)
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0, "device status word set during warm-up"
    launches = layer.sh_launch_count()

    # ---- timed region: K steps, L2 flushed before each, CUDA events on the launching stream ----
    sampler = ClockSampler(local_rank) if rank == 0 else None
    barrier()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in ev:
        flush.fill_(1)
        a.record(stream)
        layer.sh_forward(x, out)
        b.record(stream)
    barrier()
    times = np.array([a.elapsed_time(b) for a, b in ev])
    t_total_ms = float(times.sum())
    clocks = sampler.stop() if sampler else None

    # L2-warm variant: K back-to-back calls, one event pair
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record(stream)
    for _ in range(args.steps):
        layer.sh_forward(x, out)
    b.record(stream)
    torch.cuda.synchronize()
    warm_ms = a.elapsed_time(b) / args.steps

    # ---- per-stage times (CUDA events at the stage boundaries, L2 flushed) ----
    stage = np.zeros(6)
    reps = 10
    for _ in range(reps):
        flush.fill_(1)
        stage += np.array(layer.sh_forward_timed(x, out))
    stage /= reps

    # ---- end to end with host buffers: every step copies x in from pinned host memory and the
    # result back out; the three run as a pipeline on three streams (pipeline.HostFedLayer), as a
    # host-fed caller would run them ----
    from paper_2312_07987_b200 import pipeline
    xh = [x.cpu().pin_memory() for _ in range(2)]
    outh = [torch.empty(inp.x.shape, dtype=torch.float32).pin_memory() for _ in range(2)]
    pipe = pipeline.HostFedLayer(layer, x)
    for i in range(4):
        pipe.step(xh[i & 1], outh[i & 1])
    pipe.wait()
    assert torch.equal(outh[1], out.cpu()) or float((outh[1] - out.cpu()).abs().max()) < 1e-2 * float(out.abs().max()), \
        "pipelined result differs from the direct one"
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(pipe.s_in)
    for i in range(args.steps):
        pipe.step(xh[i & 1], outh[i & 1])
    b.record(pipe.s_out)
    pipe.wait()
    barrier()
    e2e_ms = a.elapsed_time(b)
    assert layer.sh_last_status() == 0, "device status word set during the timed region"

    # ---- max over ranks ----
    t_total_ms, e2e_ms, warm_ms = sharding.max_over_ranks([t_total_ms, e2e_ms, warm_ms], device="cuda")

    if rank == 0:
        N = cfg.n_tokens
        fl = inputs.useful_flop(cfg)
        ms_step = t_total_ms / args.steps
        value = sharding.aggregate_throughput(N, world, ms_step * 1e-3)
        useful_tflops = world * fl["total"] / (ms_step * 1e-3) / 1e12
        stage_flop = dict(gate_topk_sort=0.0, qk_proj=fl["qk"], v_experts=fl["v"], attention=fl["attn_half"], o_experts=fl["o"])
        dom = int(np.argmax(stage[:5]))
        dom_name = STAGES[dom]
        if dom_name == "gate_topk_sort":
            # HBM-bound stage: x read once + idx/gate/lists written
            bytes_ = N * cfg.d_model * 2 + 4 * (2 * N * cfg.n_heads * cfg.k) * 4
            ach = bytes_ / (stage[dom] * 1e-3) / 1e9
            roof = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"], traffic=None)
        else:
            ach = stage_flop[dom_name] / (stage[dom] * 1e-3) / 1e12
            roof = dict(bound="tensor", achieved=ach, peak=peaks["tflops"], unit="TFLOP/s", frac=ach / peaks["tflops"], traffic=None)
        traffic = DRAM_TRAFFIC_MB.get(cfg.name, {}).get(dom_name)
        roof.update(kernel=dom_name, ms=float(stage[dom]), peak_source=peaks["source"],
                    traffic=None if traffic is None else traffic * 1e6, traffic_unit="bytes per launch (ncu)")

        line = {
            "metric": "switchhead_layer_fwd_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == inputs.DTYPE_BF16 else "f32",
            "data": "synthetic",
            "config": {"workload": cfg.name, "batch_per_gpu": cfg.batch, "seq_len": cfg.seq, "d_model": cfg.d_model,
                       "n_heads": cfg.n_heads, "d_head": cfg.d_head, "n_experts": cfg.n_experts, "k": cfg.k,
                       "causal": True, "rope_base": args.rope if args.rope > 0 else None,
                       "shared_selection": bool(args.shared_selection),
                       "l2": "flushed before every timed step (256 MiB write)",
                       "parallelism": f"batch-sharded replicas x{world}, no collective"},
            "useful_tflops": useful_tflops,
            "frac_of_bf16_peak_measured": useful_tflops / (world * peaks["tflops"]),
            "frac_of_bf16_peak_nominal_2250": useful_tflops / (world * 2250.0),
            "ms_per_step_l2_warm": warm_ms,
            "useful_tflops_l2_warm": world * fl["total"] / (warm_ms * 1e-3) / 1e12,
            "stage_ms": {n: float(v) for n, v in zip(STAGES + ["total"], stage)},
            "gpu_launches": launches * args.steps,
            "launches_per_step": launches,
            "e2e": {"value": world * N * args.steps / (e2e_ms * 1e-3), "unit": "tokens/s",
                    "h2d_bytes_per_step": int(x.numel() * x.element_size()),
                    "d2h_bytes_per_step": int(out.numel() * 4)},
            "roofline": roof,
            "clocks": clocks,
        }
        # ---- dense multi-head comparator on the same x (262M-scale workload only) ----
        if cfg.name == "c4_262m_bf16" and not args.no_dense:
            Wq, Wk, Wv, Wo = inputs.make_dense_mha_weights(cfg.d_model, 16, 64, seed=102, dtype=cfg.dtype)
            dl = binding.Layer(cfg.d_model, 16, 64, dense=True)
            dl.sh_configure(cfg.dtype, cfg.batch, cfg.seq)
            dv = lambda t: binding.to_device(t, cfg.dtype)
            dl.sh_set_weights(dv(Wq), dv(Wk), dv(Wv[:, None]), dv(Wo[:, None]))
            for _ in range(3):
                dl.sh_forward(x, out)
            torch.cuda.synchronize()
            dt = []
            for _ in range(20):
                flush.fill_(1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream); dl.sh_forward(x, out); b.record(stream)
                torch.cuda.synchronize()
                dt.append(a.elapsed_time(b))
            dms = float(np.mean(dt))
            dense_flop = 2.0 * N * cfg.d_model * 3 * 1024 + 2.0 * cfg.batch * 16 * cfg.seq ** 2 * 64 + 2.0 * N * 1024 * cfg.d_model
            line["dense_mha_16x64"] = {"ms_per_step": dms, "switchhead_over_dense_time": ms_step / dms,
                                       "useful_tflops": dense_flop / (dms * 1e-3) / 1e12}
            dl.close()
        if not args.no_cpu_baseline:
            v, nseq, secs = oracle_sample(cfg, inp, rope_base=args.rope if args.rope > 0 else None,
                                          shared_selection=args.shared_selection)
            line["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": len(os.sched_getaffinity(0)),
                                    "kind": "oracle",
                                    "sample": f"{nseq} sequences of {cfg.seq} tokens drawn from the workload's {cfg.batch}, {secs:.1f} s, fp64 numpy"}
        line["paper_context"] = "paper reports 44% of dense MACs and 27% of dense activation memory at 262M params (analytic); no layer timing"
        print(json.dumps(line))
    layer.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
