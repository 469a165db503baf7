"""Benchmark of the PWL BERT encoder forward pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c2|c1] [--segments n]
    python bench.py --impl reference ...      # the CPU oracle, timed on the host cores

A step is one pass of the whole encoder stack (every layer: QKV GEMM, PWL attention,
out-projection + residual, PWL LayerNorm, FFN1 + PWL GELU, FFN2 + residual, PWL LayerNorm)
over one batch of seeded synthetic input.  Rank 0 prints one JSON line.

The path has no exchange step: with N > 1 every rank runs an independent replica on its own
batch (weak scaling, no collective on the data path); only the timing barrier is shared.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "PWL BERT encoder tokens/s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant (GEMM) kernel, mean over the four
# GEMM shapes of a layer, from the ncu capture summarised in profiles/encoder_c3_launches_and_kernels.md
NCU_GEMM_DRAM_BYTES_PER_LAUNCH = {"c3_bert_base_12l_bf16": 80.5e6}


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=100)
    p.add_argument("--warmup", type=int, default=10)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--workload", default="c3", choices=["c1", "c2", "c3", "c4"])
    p.add_argument("--segments", type=int, default=64)
    p.add_argument("--seed", type=int, default=0)
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--algo", type=int, default=0, help="0 auto, 1 CUDA-core kernels, 2 tensor-core kernels")
    return p.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index = index
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self.power = []
        self._stop_evt = threading.Event()
        self.error = None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                getattr(nv, "nvmlClocksEventReasonGpuIdle", 0x1): "gpu_idle",
                getattr(nv, "nvmlClocksEventReasonApplicationsClocksSetting", 0x2): "applications_clocks_setting",
                getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
                getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksEventReasonSyncBoost", 0x10): "sync_boost",
                getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
                getattr(nv, "nvmlClocksEventReasonDisplayClockSetting", 0x100): "display_clock_setting",
            }
            get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                nv.nvmlDeviceGetCurrentClocksThrottleReasons
            while not self._stop_evt.is_set():
                self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                try:
                    self.power.append(nv.nvmlDeviceGetPowerUsage(h) / 1000.0)
                except Exception:
                    pass
                mask = get_reasons(h)
                for bit, name in names.items():
                    if mask & bit and name != "gpu_idle":
                        self.reasons.add(name)
                time.sleep(0.02)
        except Exception as e:  # NVML missing: report that rather than invent clocks
            self.error = repr(e)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "error": self.error}
        s = sorted(self.samples)
        out = {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
               "samples": len(s)}
        if self.power:
            out["power_w_max"] = round(max(self.power), 1)
        return out


def dist_setup(n):
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    return world, rank, local


def physical_gpu_index(local):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except ValueError:
            return local
    return local


def oracle_tables(cfg):
    import oracle
    r = cfg.ranges()
    funcs = {"gelu": oracle.GELU, "exp": oracle.EXP, "recip": oracle.RECIP, "rsqrt": oracle.RSQRT}
    return {k: oracle.Table.secant(funcs[k], cfg.segments, *r[k]) for k in funcs}


def time_oracle(cfg, x, layers, n_layers, n_seq):
    """Times the oracle, as it stands, on `n_seq` sequences through `n_layers` layers.
    Returns (tokens/s of the FULL stack, seconds, threads)."""
    import oracle
    tabs = oracle_tables(cfg)
    L = cfg.L
    xin = x[: n_seq * L]
    t0 = time.perf_counter()
    if cfg.dtype == "i8":      # the int8 evaluation: same int8 weights and scales the GPU path receives
        import nm_inputs
        quant = nm_inputs.int8_encoder_inputs(cfg, layers[:n_layers])
        t0 = time.perf_counter()
        y = xin
        for li in range(n_layers):
            y = oracle.encoder_layer_i8(y, layers[li], quant[li], n_seq, L, cfg.heads, tabs, cfg.eps)
    else:
        oracle.encoder_stack(xin, layers[:n_layers], n_seq, L, cfg.heads, tabs, cfg.eps)
    dt = time.perf_counter() - t0
    full = dt * cfg.layers / n_layers
    return n_seq * L / full, dt, oracle.num_threads()


def run_reference(args, cfg):
    """The CPU oracle on the host cores; one step = one sequence through one layer (a bounded
    sample), scaled by the layer count to the metric's unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import nm_inputs
    import oracle
    x, layers = nm_inputs.encoder_inputs(cfg, seed=args.seed, layers=1)
    for _ in range(args.warmup):
        time_oracle(cfg, x, layers, 1, 1)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time_oracle(cfg, x, layers, 1, 1)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = cfg.L / (dt * cfg.layers)
    sample = "1 of %d sequences (%d tokens) through 1 of %d layers per step, scaled by the layer count" % (
        cfg.B, cfg.L, cfg.layers)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(cfg, args):
    return {"workload": cfg.name, "layers": cfg.layers, "batch": cfg.B, "seq_len": cfg.L, "hidden": cfg.H,
            "heads": cfg.heads, "ffn": cfg.F, "pwl_segments": cfg.segments, "seed": args.seed,
            "parallelism": "replicas" if args.gpus > 1 else "single",
            "l2": "working set per step (weights %.0f MB + activations %.0f MB) exceeds the 126 MB L2; no flush"
                  % (cfg.layers * (4 * cfg.H * cfg.H + 2 * cfg.H * cfg.F) * 2 / 1e6,
                     cfg.T * (6 * cfg.H + cfg.F) * 2 / 1e6)}


def main():
    args = parse_args()
    import nm_inputs
    cfg = nm_inputs.with_(nm_inputs.CONFIGS[args.workload], segments=args.segments)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    import paper_2305_14405_b200 as nm
    from paper_2305_14405_b200.harness import EncoderModel

    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    world, rank, local = dist_setup(args.gpus)
    dev = "cuda:%d" % local
    torch.cuda.set_device(local)
    nm.load()
    ctx = nm.Context(local)
    ctx.load_encoder_tables(cfg.segments, cfg.ranges())
    # every rank draws its own batch (seed + rank): independent replicas of the same model
    x_np, layers_np = nm_inputs.encoder_inputs(cfg, seed=args.seed)
    if rank > 0:
        x_np, _ = nm_inputs.encoder_inputs(cfg, seed=args.seed + rank, layers=0)
    quant = nm_inputs.int8_encoder_inputs(cfg, layers_np) if cfg.dtype == "i8" else None
    model = EncoderModel(ctx, cfg, layers_np, device=dev, algo=args.algo, quant=quant)
    act = model.act_dtype()
    x = torch.from_numpy(x_np).to(dev).to(act)
    y = torch.empty_like(x)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        model.forward(x, y)
    ctx.check_device_status()

    # ---- timed region: K steps, CUDA events on the launching stream ------------------------
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    time.sleep(0.05)
    ev0 = torch.cuda.Event(enable_timing=True)
    ev1 = torch.cuda.Event(enable_timing=True)
    ctx.launch_count(reset=True)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        model.forward(x, y)
    ev1.record(stream)
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    launches = ctx.launch_count()
    sampler.stop()
    ctx.check_device_status()
    t = torch.tensor([ms_total], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_total = float(t.item())
    ms_step = ms_total / args.steps
    value = world * cfg.T / (ms_step * 1e-3)

    # ---- per-kernel pass: the same steps with every launch bracketed by events -------------
    prof_steps = min(args.steps, max(1, 8000 // max(1, launches // max(args.steps, 1))))
    ctx.profile_enable(True)
    for _ in range(prof_steps):
        model.forward(x, y)
    torch.cuda.synchronize()
    prof = ctx.profile_read()
    ctx.profile_enable(False)

    # ---- end to end through the C ABI with host buffers ------------------------------------
    xh = torch.from_numpy(x_np).to(act).pin_memory()
    yh = torch.empty_like(xh).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))
    ctx.encoder_stack_host(model.array, model.n_layers, model.ccfg, xh, yh, x, y, model.workspace)
    barrier()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        ctx.encoder_stack_host(model.array, model.n_layers, model.ccfg, xh, yh, x, y, model.workspace)
    e1.record(stream)
    barrier()
    t = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    e2e_ms = float(t.item()) / e2e_steps
    act_bytes = cfg.T * cfg.H * x.element_size()

    if rank == 0:
        peaks, peak_kind = load_peaks()
        total_ms = sum(v[1] for v in prof.values()) or 1.0
        kernels = {k: {"launches_per_step": v[0] / prof_steps, "ms_per_step": v[1] / prof_steps,
                       "share": v[1] / total_ms} for k, v in prof.items() if v[0]}
        gemm_kind = "linear_tc" if prof["linear_tc"][0] else "linear_simt"
        n_l, ms_l, work_l = prof[gemm_kind]
        achieved = work_l / (ms_l * 1e-3) / 1e12 if ms_l > 0 else 0.0
        # int8: the measured bf16 peak times the nominal 2:1 int8:bf16 ratio; fp32 runs on CUDA cores
        peak = {"i8": 2.0, "f32": 0.5}.get(cfg.dtype, 1.0) * peaks["bf16_tflops_sustained"]
        roofline = {"bound": "tensor", "kernel": gemm_kind, "achieved": achieved, "peak": peak,
                    "unit": "TFLOP/s", "frac": achieved / peak,
                    "traffic": NCU_GEMM_DRAM_BYTES_PER_LAUNCH.get(cfg.name),
                    "peak_source": "%s (bf16 sustained: kernel timed inside a long step)" % peak_kind,
                    "avg_launch_us": ms_l / max(n_l, 1) * 1e3, "share_of_step": ms_l / total_ms}
        extra = {}
        n_ln, ms_ln, work_ln = prof["layernorm"]
        if n_ln:
            gbs = work_ln / (ms_ln * 1e-3) / 1e9
            extra["layernorm"] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                  "frac": gbs / peaks["hbm_gbs"], "note": "algorithmic bytes; input is L2-resident "
                                  "after the producing GEMM at this size"}
        for kind in ("attention_tc", "attention_simt"):
            n_a, ms_a, work_a = prof[kind]
            if n_a:
                tf = work_a / (ms_a * 1e-3) / 1e12
                extra[kind] = {"bound": "alu", "achieved_tensor_tflops": tf, "avg_launch_us": ms_a / n_a * 1e3}
        whole = cfg.layers * cfg.flops_per_layer() / (ms_step * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic", "config": workload_config(cfg, args),
            "clocks": sampler.summary(),
            "e2e": {"value": world * cfg.T / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": act_bytes,
                    "d2h_bytes_per_step": act_bytes, "ms_per_step": e2e_ms},
            "gpu_launches": launches,
            "roofline": roofline,
            "roofline_other": extra,
            "kernels": kernels,
            "whole_step_tflops": whole,
        }
        if not args.no_cpu_baseline and world == 1:
            # calibrate on one sequence through one layer, then size the sample to ~15 s of CPU work
            _, t1, _ = time_oracle(cfg, x_np, layers_np, 1, 1)
            n_layers = max(1, min(cfg.layers, int(15.0 / max(t1, 1e-3))))
            n_seq = max(1, min(cfg.B, int(15.0 / max(t1 * n_layers, 1e-3))))
            v, secs, cores = time_oracle(cfg, x_np, layers_np, n_layers, n_seq)
            line["cpu_baseline"] = {
                "value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": "%d of %d sequences (%d tokens each) through %d of %d layers, %.1f s%s"
                          % (n_seq, cfg.B, cfg.L, n_layers, cfg.layers, secs,
                             "" if n_layers == cfg.layers else "; scaled by the layer count")}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    ctx.close()


if __name__ == "__main__":
    main()
