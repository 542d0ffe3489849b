#!/usr/bin/env python
"""Benchmark of the fused block-scaled FP8 MoE forward (one B200 per rank).

A step = one whole forward pass (routing, permutation, GEMM1+SwiGLU+requant,
GEMM2, combine) over one batch of synthetic tokens.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config i] [--impl reference]

N > 1 is launched under torch.distributed.run; every rank runs an independent
replica of the layer on its own batch (no data-path collective, weak scaling).
`--impl reference` times the CPU oracle (a deliberately plain program) on the
same workload, on rank 0 only.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_14560_b200 import synthetic as syn  # noqa: E402

FLOPS_PER_SLOT = 2 * 7168 * 4096 + 2 * 2048 * 7168            # 88 080 384
BYTES_PER_EXPERT = 4096 * 7168 + 7168 * 2048 + 32 * 56 * 4 + 56 * 16 * 4  # weights + their scales
W13_BYTES_PER_EXPERT = 4096 * 7168 + 32 * 56 * 4
W2_BYTES_PER_EXPERT = 7168 * 2048 + 56 * 16 * 4
FP8_DATASHEET_TFLOPS = 4500.0
HBM_DATASHEET_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the committed ncu capture of the headline
# workload (profiles/launches_dsv3_T64_E32.md), mean over the two rotating activation sets.
NCU_TRAFFIC_BYTES = {
    ("dsv3_T64_E32", "gemm1_swiglu_quant"): (486.1e6 + 4.4e6 + 455.7e6 + 0.7e6) / 2,
    ("dsv3_T64_E32", "gemm2"): (239.5e6 + 3.2e6 + 224.5e6 + 2.6e6) / 2,
}
METRIC = "fused FP8 MoE forward throughput (tokens/s; TFLOPS and roofline fraction alongside)"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value: float, world: int, device=None) -> float:
    """MAX all-reduce of a scalar (nccl on GPU tensors, gloo on CPU tensors)."""
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, world: int, device=None) -> float:
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.stop_flag, self.mhz, self.reasons, self.max_mhz = index, False, [], set(), None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            }
            while not self.stop_flag:
                self.mhz.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
                time.sleep(0.002)
        except Exception as ex:  # clocks are reported as unknown, the run itself is unaffected
            self.reasons.add(f"nvml_unavailable:{type(ex).__name__}")

    def result(self):
        return {"sm_mhz": statistics.median(self.mhz) if self.mhz else None, "sm_max_mhz": self.max_mhz,
                "samples": len(self.mhz), "reasons": sorted(self.reasons)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# --------------------------------------------------------------------------
# CUDA arm
# --------------------------------------------------------------------------
def routing_stats(eng, T, dims, offset):
    dbg = eng.debug_export(T, rows=False)
    torch.cuda.synchronize()
    cnt = dbg["expert_count"].cpu().numpy()
    return int(cnt.sum()), int((cnt > 0).sum()), int(dbg["status"].item())


def time_steps(eng, weights, acts, outs, flush, steps, stage=False):
    """Times `steps` forwards with CUDA events on the launching stream; an L2 flush
    (untimed) precedes each step and the activation sets are rotated.  The flush
    writes one buffer larger than L2 and then reads a second one: the read pushes
    the dirty lines of the write out, so their write-back to HBM does not land
    inside the timed region (it cost the first GEMM about 15 % of its bandwidth)."""
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    stage_ms = []
    for i in range(steps):
        a = acts[i % len(acts)]
        flush[0].zero_()
        flush[1].view(torch.int64).sum()
        ev[i][0].record()
        eng.forward({**weights, **a}, out=outs[i % len(outs)])
        ev[i][1].record()
        if stage:
            stage_ms.append(eng.get_stage_times())
    torch.cuda.synchronize()
    total = sum(s.elapsed_time(e) for s, e in ev)
    return total, stage_ms


def run_cuda_config(wl, device, steps, warmup, peaks, peak_kind, want_e2e=True, cpu_baseline=False,
                    sampler_index=None):
    from paper_2608_14560_b200 import MoeFp8
    d = wl.dims
    T = wl.tokens
    inp = syn.make_inputs(wl, device)
    weights = {k: inp[k] for k in ("routing_bias", "w13", "w13_scale", "w2", "w2_scale", "local_expert_offset",
                                   "scaling_factor")}
    acts = [{k: inp[k] for k in ("hidden_fp8", "hidden_scale", "router_logits")},
            syn.make_activations(wl, wl.seed + 1000, device)]
    outs = [torch.empty(T, d.hidden, dtype=torch.bfloat16, device=device) for _ in range(2)]
    flush = [torch.zeros(256 << 20, dtype=torch.uint8, device=device) for _ in range(2)]
    eng = MoeFp8(d.hidden, d.intermediate, d.num_experts, d.num_local_experts, d.n_group, d.topk_group, d.top_k,
                 max_tokens=T, device=device)

    per_set = []
    for a in acts:  # real slot / active-expert counts of each activation set
        eng.forward({**weights, **a}, out=outs[0])
        per_set.append(routing_stats(eng, T, d, wl.local_expert_offset))
    assert all(s[2] == 0 for s in per_set), f"device status {per_set}"
    S = float(np.mean([s[0] for s in per_set]))
    A = float(np.mean([s[1] for s in per_set]))

    time_steps(eng, weights, acts, outs, flush, max(warmup, 3))
    sampler = ClockSampler(sampler_index) if sampler_index is not None else None
    if sampler:
        sampler.start()
    world = dist_env()[2]
    if world > 1:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    total_ms, _ = time_steps(eng, weights, acts, outs, flush, steps)
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
    launches = eng.last_launch_count() * steps
    status = eng.status()
    assert status == 0, f"device status {status} after the timed region"

    # per-kernel device times over the same kind of region (events around every launch)
    eng.set_stage_timing(True)
    time_steps(eng, weights, acts, outs, flush, 3, stage=True)
    _, stage_ms = time_steps(eng, weights, acts, outs, flush, steps, stage=True)
    eng.set_stage_timing(False)
    if sampler:  # clocks are sampled across the timed region and the identical per-kernel pass
        sampler.stop_flag = True
        sampler.join()
    stage_avg = {k: float(np.mean([s[k] for s in stage_ms])) for k in stage_ms[0]}

    ms = total_ms / steps
    flops = FLOPS_PER_SLOT * S * (d.hidden * d.intermediate) / (7168 * 2048)
    t_flop = flops / (FP8_DATASHEET_TFLOPS * 1e12)
    t_hbm = BYTES_PER_EXPERT * A / (HBM_DATASHEET_GBS * 1e9)
    bound = "tensor" if t_flop > t_hbm else "hbm"
    res = {
        "workload": wl.name, "tokens": T, "local_slots": S, "active_experts": A, "ms_per_step": ms,
        "tokens_per_s": T / (ms * 1e-3), "tflops": flops / (ms * 1e-3) / 1e12,
        "weight_gbs": BYTES_PER_EXPERT * A / (ms * 1e-3) / 1e9,
        "roofline_bound": bound, "roofline_frac_of_datasheet": max(t_flop, t_hbm) / (ms * 1e-3),
        "stage_ms": stage_avg, "launches_per_step": eng.last_launch_count(), "total_ms": total_ms,
        "gpu_launches": launches,
    }
    # roofline of the dominant kernel, against the measured peaks of this machine
    dom = max(stage_avg, key=stage_avg.get)
    dom_s = stage_avg[dom] * 1e-3
    g1_flops = 2 * d.hidden * 2 * d.intermediate * S
    g2_flops = 2 * d.intermediate * d.hidden * S
    kern_flops = {"gemm1_swiglu_quant": g1_flops, "gemm2": g2_flops}.get(dom, 0.0)
    kern_bytes = {"gemm1_swiglu_quant": W13_BYTES_PER_EXPERT * A + S * (d.hidden + d.hidden // 32 + d.intermediate),
                  "gemm2": W2_BYTES_PER_EXPERT * A + S * (d.intermediate + 2 * d.hidden)}.get(dom, 0.0)
    fp8_peak = 2.0 * peaks["bf16_tflops_sustained" if ms * steps > 500 else "bf16_tflops"]
    if kern_flops / (fp8_peak * 1e12) > kern_bytes / (peaks["hbm_gbs"] * 1e9):
        ach = kern_flops / dom_s / 1e12
        res["roofline"] = {"bound": "tensor", "kernel": dom, "achieved": ach, "peak": fp8_peak, "unit": "TFLOP/s",
                           "frac": ach / fp8_peak, "traffic": None,
                           "peak_source": f"2 x {peak_kind} bf16 cuBLAS peak (fp8:bf16 nominal ratio 2)"}
    else:
        ach = kern_bytes / dom_s / 1e9
        res["roofline"] = {"bound": "hbm", "kernel": dom, "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                           "frac": ach / peaks["hbm_gbs"], "traffic": None, "peak_source": f"{peak_kind} copy bandwidth"}
    res["roofline"]["traffic"] = NCU_TRAFFIC_BYTES.get((wl.name, dom))
    res["roofline"]["algorithmic_per_launch"] = kern_flops if res["roofline"]["bound"] == "tensor" else kern_bytes
    res["roofline"]["kernel_ms"] = stage_avg[dom]
    if sampler:
        res["clocks"] = sampler.result()

    if want_e2e:
        host_acts = [{k: v.cpu().pin_memory() for k, v in a.items()} for a in acts]
        host_out = torch.empty(T, d.hidden, dtype=torch.bfloat16).pin_memory()
        for i in range(3):
            eng.forward_host(host_acts[i % 2], weights, host_out)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(steps):
            eng.forward_host(host_acts[i % 2], weights, host_out)
        e2e_s = (time.perf_counter() - t0) / steps
        h2d = sum(v.numel() * v.element_size() for v in host_acts[0].values())
        res["e2e"] = {"value": T / e2e_s, "unit": "tokens/s", "ms_per_step": e2e_s * 1e3,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": host_out.numel() * 2,
                      "checksum": float(host_out.float().abs().sum())}

    if cpu_baseline:
        res["cpu_baseline"] = oracle_baseline(wl, syn.to_host(inp))
    eng.close()
    del eng, inp, weights, acts, outs
    torch.cuda.empty_cache()
    return res


# --------------------------------------------------------------------------
# CPU oracle arm (the reported baseline; test infrastructure, never tuned)
# --------------------------------------------------------------------------
def oracle_sample_tokens(wl, budget_slots=400):
    """A bounded sample of the workload: as many leading tokens as ~budget_slots
    (token, expert) slots at ~22 ms of single-thread CPU time each."""
    per_token = 8.0 * wl.dims.num_local_experts / wl.dims.num_experts
    if wl.skew:
        per_token = 4.5
    n = int(max(1, min(wl.tokens, budget_slots / max(per_token, 0.25))))
    return np.arange(n, dtype=np.int32)


def oracle_baseline(wl, host, min_seconds=10.0):
    """The oracle as it stands, one thread, on a bounded token sample, repeated until ~10 s of CPU work."""
    import oracle
    d = wl.dims
    tokens = oracle_sample_tokens(wl)
    t0 = time.perf_counter()
    reps = 0
    while True:
        oracle.forward(host, d.n_group, d.topk_group, d.top_k, tokens=tokens)
        reps += 1
        if time.perf_counter() - t0 >= min_seconds or reps >= 64:
            break
    total = time.perf_counter() - t0
    dt = total / reps
    return {"value": len(tokens) / dt, "unit": "tokens/s", "cores": 1, "kind": "oracle",
            "sample": f"first {len(tokens)} of {wl.tokens} tokens of {wl.name} (routing on all tokens), "
                      f"single thread, {reps} pass(es), {total:.1f} s in total", "host_cores": os.cpu_count()}


def run_reference(args, wl):
    import oracle
    d = wl.dims
    host = syn.to_host(syn.make_inputs(wl, "cuda:0" if torch.cuda.is_available() else "cpu"))
    # Each step is a bounded sample, sized so that steps + warm-up end within about two and a half minutes
    # at ~22 ms of single-thread CPU time per (token, expert) slot.
    per_step_s = 150.0 / (args.steps + max(args.warmup, 1))
    tokens = oracle_sample_tokens(wl, budget_slots=max(1.0, min(120.0, per_step_s / 0.022)))
    for _ in range(max(args.warmup, 1)):
        oracle.forward(host, d.n_group, d.topk_group, d.top_k, tokens=tokens[: max(1, len(tokens) // 8)])
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.forward(host, d.n_group, d.topk_group, d.top_k, tokens=tokens)
    dt = (time.perf_counter() - t0) / args.steps
    v = len(tokens) / dt
    sample = f"each step = first {len(tokens)} of {wl.tokens} tokens of {wl.name}, single thread"
    return {
        "impl": "reference", "metric": METRIC, "value": v, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3 x fp8_e4m3 -> f32",
        "data": "synthetic",
        "config": {"workload": wl.name, "tokens_per_gpu": wl.tokens, "hidden": d.hidden, "intermediate": d.intermediate,
                   "local_experts": d.num_local_experts, "sample": sample,
                   "stands_in_for": "FlashInfer-Bench Fused-MoE contest workloads (DeepSeek-V3 shapes)"},
        "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


# --------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=1, help="index into the five benchmark workloads (headline)")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--others", default="0,2,3,4", help="extra workloads reported under 'workloads' at N=1 ('' = none)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--tokens", type=int, default=0, help="override T of the chosen workload (profiling runs)")
    ap.add_argument("--paper-points", default="7,54,14107",
                    help="token counts the paper quotes a latency for (its table of workload regimes: short / median / long); "
                         "timed on the 32-local-expert layer and reported under 'paper_points' ('' = none)")
    args = ap.parse_args()
    rank, local_rank, world = dist_env()
    wl = syn.CONFIGS[args.config]
    if args.tokens > 0:
        wl = syn.Workload(f"{wl.name}_T{args.tokens}", args.tokens, wl.dims, wl.seed, wl.local_expert_offset,
                          wl.scaling_factor, wl.skew)

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args, wl)), flush=True)
        return 0

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a B200: the CUDA path has no CPU fallback")
    device = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(device)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    peaks, peak_kind = load_peaks()

    my_wl = syn.Workload(wl.name, wl.tokens, wl.dims, wl.seed + 7919 * rank, wl.local_expert_offset,
                         wl.scaling_factor, wl.skew)
    res = run_cuda_config(my_wl, device, args.steps, args.warmup, peaks, peak_kind, want_e2e=not args.no_e2e,
                          cpu_baseline=(rank == 0 and world == 1 and not args.no_cpu_baseline),
                          sampler_index=physical_gpu_index(local_rank))
    total_ms = max_over_ranks(res["total_ms"], world, device)
    if args.no_e2e:
        res["e2e"] = {"ms_per_step": float("nan"), "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    e2e_ms = max_over_ranks(res["e2e"]["ms_per_step"], world, device)
    tokens_all = sum_over_ranks(float(my_wl.tokens), world, device)
    launches = sum_over_ranks(float(res["gpu_launches"]), world, device)

    others = []
    if world == 1 and args.others:
        for i in [int(x) for x in args.others.split(",") if x != ""]:
            if i == args.config:
                continue
            w = syn.CONFIGS[i]
            st = args.steps if w.tokens <= 1024 else max(5, args.steps // 5)
            r = run_cuda_config(w, device, st, max(3, args.warmup), peaks, peak_kind, want_e2e=False,
                                sampler_index=physical_gpu_index(local_rank))
            r.pop("total_ms")
            others.append(r)

    # The paper's three quoted latencies (B200, 32 local experts of 256, contest workloads whose routing is not
    # published): the same token counts on the synthetic layer of workload 1, as context.
    paper_ms = {7: 0.099, 54: 0.205, 14107: 1.229}
    points = []
    if world == 1 and args.paper_points:
        base = syn.CONFIGS[1]
        for t in [int(x) for x in args.paper_points.split(",") if x != ""]:
            w = syn.Workload(f"dsv3_T{t}_E32", t, base.dims, base.seed, base.local_expert_offset,
                             base.scaling_factor, base.skew)
            st = args.steps if t <= 1024 else max(5, args.steps // 5)
            r = run_cuda_config(w, device, st, max(3, args.warmup), peaks, peak_kind, want_e2e=False)
            points.append({"tokens": t, "ms_per_step": r["ms_per_step"], "paper_ms": paper_ms.get(t),
                           "local_slots": r["local_slots"], "active_experts": r["active_experts"],
                           "tflops": r["tflops"], "weight_gbs": r["weight_gbs"]})

    if rank == 0:
        ms = total_ms / args.steps
        line = {
            "metric": METRIC,
            "value": tokens_all / (ms * 1e-3), "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp8_e4m3 x fp8_e4m3 -> f32", "data": "synthetic",
            "config": {"workload": wl.name, "tokens_per_gpu": wl.tokens, "hidden": wl.dims.hidden,
                       "intermediate": wl.dims.intermediate, "local_experts": wl.dims.num_local_experts,
                       "local_slots": res["local_slots"], "active_experts": res["active_experts"],
                       "parallelism": f"{world} independent replica(s), no collective",
                       "l2": "untimed flush between timed iterations: a 256 MiB buffer is written, then a second 256 MiB buffer is read so that no dirty lines are left; two rotating activation sets",
                       "stands_in_for": "FlashInfer-Bench Fused-MoE contest workloads (DeepSeek-V3 shapes)"},
            "tflops": res["tflops"] * world, "weight_gbs_per_gpu": res["weight_gbs"],
            "roofline_frac_of_datasheet": {"bound": res["roofline_bound"], "frac": res["roofline_frac_of_datasheet"],
                                           "fp8_tflops": FP8_DATASHEET_TFLOPS, "hbm_gbs": HBM_DATASHEET_GBS},
            "roofline": res["roofline"], "stage_ms": res["stage_ms"],
            "e2e": {"value": tokens_all / (e2e_ms * 1e-3), "unit": "tokens/s",
                    "h2d_bytes_per_step": res["e2e"]["h2d_bytes_per_step"],
                    "d2h_bytes_per_step": res["e2e"]["d2h_bytes_per_step"], "ms_per_step": e2e_ms},
            "gpu_launches": int(launches), "clocks": res.get("clocks"),
            "cpu_baseline": res.get("cpu_baseline"), "peaks": peak_kind, "workloads": others,
            "paper_points": points,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
