"""Benchmark of the PWL forward pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c2|c1|c4|c5|rows] [--segments n]
    python bench.py --impl reference ...      # the CPU oracle, timed on the host cores

Default workload c3: the 12-layer BERT-base-shaped PWL encoder (batch 32, seq 512), the
configuration the metric "PWL BERT encoder tokens/s" is quoted on.  A step is one pass of the whole
network over one batch of seeded synthetic input (encoder: per layer QKV GEMM, PWL attention,
out-projection + residual, PWL LayerNorm, FFN1 + PWL GELU, FFN2 + residual, PWL LayerNorm; c5: the
ResNet-50-shaped CNN, 53 convolutions as GEMMs with ReLU tables, pools, classifier).  Rank 0 prints
one JSON line.

The path has no exchange step: with N > 1 every rank runs an independent replica on its own batch
(weak scaling, no collective on the data path); only the timing barrier is shared.
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

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_BF16_TFLOPS = 2250.0      # dense bf16 / fp16 tensor peak of the part, for context
NOMINAL_HBM_GBS = 8000.0
REPEATS = 5                       # the K-step timed region is repeated; value = median over the repeats


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=100)
    p.add_argument("--warmup", type=int, default=10)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--workload", default="c3", choices=["c1", "c2", "c3", "c4", "c5", "rows"])
    p.add_argument("--segments", type=int, default=64)
    p.add_argument("--seed", type=int, default=0)
    p.add_argument("--batch", type=int, default=0, help="override the batch size (c5 only)")
    p.add_argument("--ln-two-table", action="store_true",
                   help="rows workload: LayerNorm as PWL_recip(PWL_sqrt(v + eps)) instead of one rsqrt table")
    p.add_argument("--hidden", type=int, default=0, help="encoder workloads: override H (heads = H/64, F = 4H)")
    p.add_argument("--layers", type=int, default=0, help="encoder workloads: override the number of layers")
    p.add_argument("--resnet-blocks", default="", help="c5: bottleneck blocks per stage, e.g. 3,4,23,3 (default 3,4,6,3)")
    p.add_argument("--resnet-width", type=int, default=0, help="c5: width of the first stage (default 64)")
    p.add_argument("--calibrated", action="store_true",
                   help="encoder workloads: table ranges observed by running the exact model (tests/golden/calibrated_ranges.json)")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-other-legs", action="store_true",
                   help="default c3 line: skip the short c4 (int8 encoder) and c5 (CNN) passes reported under other_workloads")
    p.add_argument("--no-rows-leg", action="store_true",
                   help="encoder workloads: skip the row-kernel bandwidth leg on a tensor beyond L2")
    p.add_argument("--repeats", type=int, default=REPEATS, help="how many times the K-step timed region is run")
    p.add_argument("--streams", type=int, default=2, choices=[1, 2, 3, 4],
                   help="steps in flight: n > 1 = the K steps rotate over n streams, each with its own buffers")
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
        self.reason_samples = {}
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
            names = {0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
                     0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
                     0x100: "display_clock_setting"}
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
                    if mask & bit:
                        self.reasons.add(name)
                        self.reason_samples[name] = self.reason_samples.get(name, 0) + 1
                time.sleep(0.005)
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
               "samples": len(s), "sm_mhz_min": s[0], "reason_samples": dict(self.reason_samples)}
        if self.power:
            out["power_w_max"] = round(max(self.power), 1)
        return out


def dist_setup():
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


# ----------------------------------------------------------------------------------------------
# workloads
# ----------------------------------------------------------------------------------------------

def fork_streams(wl, stream):
    """Two slots (device input, device output, workspace, pinned result, stream) for steps in flight together;
    slot 0 is the workload's own buffers.  Both streams are ordered after what `stream` holds."""
    import torch
    if not hasattr(wl, "slots"):
        ws = wl.model.workspace
        wl.slots = [(wl.x, wl.y, ws, wl.yh, torch.cuda.Stream())]
        for _ in range(1, max(2, wl.args.streams)):
            wl.slots.append((wl.x.clone(), torch.empty_like(wl.y), torch.empty_like(ws),
                             torch.empty_like(wl.yh).pin_memory(), torch.cuda.Stream()))
        torch.cuda.synchronize()
    start = torch.cuda.Event()
    start.record(stream)
    for sl in wl.slots:
        sl[4].wait_event(start)


def join_streams(wl, stream):
    """`stream` waits for everything the two slot streams hold."""
    import torch
    for sl in wl.slots:
        done = torch.cuda.Event()
        done.record(sl[4])
        stream.wait_event(done)


class EncoderWorkload:
    """c1..c4: the PWL transformer encoder stack; unit = tokens."""
    metric = "PWL BERT encoder tokens/s"
    unit = "tokens/s"

    def __init__(self, args):
        import nm_inputs
        self.args = args
        self.cfg = nm_inputs.with_(nm_inputs.CONFIGS[args.workload], segments=args.segments)
        if args.hidden or args.layers:   # width / depth sweep: same recipe, other shape
            H = args.hidden or self.cfg.H
            assert H % 64 == 0, "--hidden must be a multiple of the head size 64"
            self.cfg = nm_inputs.with_(self.cfg, H=H, heads=H // 64, F=4 * H, layers=args.layers or self.cfg.layers,
                                       name="%s_H%d_L%d" % (self.cfg.name, H, args.layers or self.cfg.layers))
        self.dtype = self.cfg.dtype
        self.units_per_step = self.cfg.T

    def config(self, world):
        c = self.cfg
        return {"workload": c.name, "layers": c.layers, "batch": c.B, "seq_len": c.L, "hidden": c.H, "heads": c.heads,
                "ffn": c.F, "pwl_segments": c.segments, "seed": self.args.seed,
                "table_ranges": "calibrated" if self.args.calibrated else "fixed",
                "parallelism": "replicas" if world > 1 else "single",
                "l2": "working set per step (weights %.0f MB + activations %.0f MB) exceeds the 126 MB L2; no flush"
                      % (c.layers * (4 * c.H * c.H + 2 * c.H * c.F) * (1 if c.dtype == "i8" else 2) / 1e6,
                         c.T * (6 * c.H + c.F) * 2 / 1e6)}

    def flops_per_step(self):
        return self.cfg.layers * self.cfg.flops_per_layer()

    def setup(self, ctx, dev, rank):
        import torch
        import nm_inputs
        from paper_2305_14405_b200.harness import EncoderModel
        cfg = self.cfg
        ctx.load_encoder_tables(cfg.segments, cfg.ranges(self.args.calibrated))
        self.x_np, self.layers_np = nm_inputs.encoder_inputs(cfg, seed=self.args.seed)
        if rank > 0:  # every rank draws its own batch: independent replicas of the same model
            self.x_np, _ = nm_inputs.encoder_inputs(cfg, seed=self.args.seed + rank, layers=0)
        quant = nm_inputs.int8_encoder_inputs(cfg, self.layers_np) if cfg.dtype == "i8" else None
        self.model = EncoderModel(ctx, cfg, self.layers_np, device=dev, algo=self.args.algo, quant=quant)
        act = self.model.act_dtype()
        self.x = torch.from_numpy(self.x_np).to(dev).to(act)
        self.y = torch.empty_like(self.x)
        self.xh = torch.from_numpy(self.x_np).to(act).pin_memory()
        self.yh = torch.empty_like(self.xh).pin_memory()
        self.ctx = ctx
        self.h2d = self.d2h = cfg.T * cfg.H * self.x.element_size()

    def step(self):
        self.model.forward(self.x, self.y)

    def host_step(self):
        m = self.model
        self.ctx.encoder_stack_host(m.array, m.n_layers, m.ccfg, self.xh, self.yh, self.x, self.y, m.workspace)

    e2e_pipeline = "one stream per step in flight (--streams), each with its own device buffers, workspace and pinned result buffer"

    def host_steps(self, k, stream):
        """k calls of nm_encoder_stack_host_async, alternating between two streams: the copies of one call
        overlap the kernels of the other.  Everything is ordered after what `stream` holds, and `stream`
        waits for both at the end."""
        m = self.model
        fork_streams(self, stream)
        for i in range(k):
            x, y, ws, yh, st = self.slots[i % len(self.slots)]
            self.ctx.encoder_stack_host(m.array, m.n_layers, m.ccfg, self.xh, yh, x, y, ws, stream=st, wait=False)
        join_streams(self, stream)

    def device_steps(self, k, stream):
        """k steps on device-resident inputs, alternating between the two streams (independent batches: the
        ramp and drain of one step's kernels overlap the other's)."""
        m = self.model
        fork_streams(self, stream)
        for i in range(k):
            x, y, ws, yh, st = self.slots[i % len(self.slots)]
            self.ctx.encoder_stack(m.array, m.n_layers, m.ccfg, x, y, ws, stream=st)
        join_streams(self, stream)

    # -- the oracle, as it stands, on whole sampled sequences (sequences are independent) -----------
    def _oracle_tables(self):
        import oracle
        r = self.cfg.ranges(self.args.calibrated)
        funcs = {"gelu": oracle.GELU, "exp": oracle.EXP, "recip": oracle.RECIP, "rsqrt": oracle.RSQRT}
        return {k: oracle.Table.secant(funcs[k], self.cfg.segments, *r[k]) for k in funcs}

    def time_oracle(self, x, layers, n_layers, n_seq):
        """Returns (units/s of the FULL stack, seconds, threads)."""
        import oracle
        cfg = self.cfg
        tabs = self._oracle_tables()
        xin = x[: n_seq * cfg.L]
        if cfg.dtype == "i8":  # the int8 evaluation: same int8 weights and scales the GPU path receives
            import nm_inputs
            quant = nm_inputs.int8_encoder_inputs(cfg, layers[:n_layers])
            t0 = time.perf_counter()
            y = xin
            for li in range(n_layers):
                y = oracle.encoder_layer_i8(y, layers[li], quant[li], n_seq, cfg.L, cfg.heads, tabs, cfg.eps)
        else:
            t0 = time.perf_counter()
            oracle.encoder_stack(xin, layers[:n_layers], n_seq, cfg.L, cfg.heads, tabs, cfg.eps)
        dt = time.perf_counter() - t0
        return n_seq * cfg.L / (dt * cfg.layers / n_layers), dt, oracle.num_threads()

    def cpu_baseline(self):
        cfg = self.cfg
        _, t1, _ = self.time_oracle(self.x_np, self.layers_np, 1, 1)   # calibrate, then ~15 s of CPU work
        n_layers = max(1, min(cfg.layers, int(15.0 / max(t1, 1e-3))))
        n_seq = max(1, min(cfg.B, int(15.0 / max(t1 * n_layers, 1e-3))))
        v, secs, cores = self.time_oracle(self.x_np, self.layers_np, n_layers, n_seq)
        return {"value": v, "unit": self.unit, "cores": cores, "kind": "oracle",
                "sample": "%d of %d sequences (%d tokens each) through %d of %d layers, %.1f s%s"
                          % (n_seq, cfg.B, cfg.L, n_layers, cfg.layers, secs,
                             "" if n_layers == cfg.layers else "; scaled by the layer count")}

    def reference_setup(self):
        import nm_inputs
        self.x_np, self.layers_np = nm_inputs.encoder_inputs(self.cfg, seed=self.args.seed, layers=1)
        self.ref_sample = "1 of %d sequences (%d tokens) through 1 of %d layers per step, scaled by the layer count" % (
            self.cfg.B, self.cfg.L, self.cfg.layers)

    def reference_step(self):
        """Runs one bounded sample; returns the units of full-network work it stands for."""
        self.time_oracle(self.x_np, self.layers_np, 1, 1)
        return self.cfg.L / self.cfg.layers


class ResnetWorkload:
    """c5: the ResNet-50-shaped CNN run as GEMMs with ReLU tables, fp16 NHWC; unit = images."""
    metric = "PWL ResNet-50 images/s"
    unit = "images/s"
    dtype = "f16"

    def __init__(self, args):
        self.args = args
        self.batch = args.batch or 128
        self.units_per_step = self.batch
        self.blocks = tuple(int(v) for v in args.resnet_blocks.split(",")) if args.resnet_blocks else (3, 4, 6, 3)
        assert len(self.blocks) == 4, "--resnet-blocks takes four numbers"
        self.base = args.resnet_width or 64
        self.variant = self.blocks != (3, 4, 6, 3) or self.base != 64

    def config(self, world):
        name = "c5_resnet50_f16" if not self.variant else "c5_resnet_b%s_w%d_f16" % ("-".join(map(str, self.blocks)), self.base)
        return {"workload": name, "batch": self.batch, "image": "224x224x3 NHWC",
                "blocks": list(self.blocks), "base_width": self.base, "convolutions": 1 + sum(3 * b + 1 for b in self.blocks),
                "classes": 1000, "batchnorm": "folded into weights and biases", "relu": "2-segment PWL table",
                "seed": self.args.seed, "parallelism": "replicas" if world > 1 else "single",
                "l2": "activations (up to %.0f MB per layer at this batch) exceed the 126 MB L2; no flush"
                      % (self.batch * 112 * 112 * self.base * 2 / 1e6)}

    def flops_per_step(self):
        import nm_inputs_cnn
        specs = iter(nm_inputs_cnn.resnet_conv_specs(self.blocks, self.base))
        cin, cout, k, _, _ = next(specs)
        total = 2 * 112 * 112 * cout * k * k * cin
        h = 56
        for st, nb in enumerate(self.blocks):
            for b in range(nb):
                stride = 2 if (b == 0 and st > 0) else 1
                ho = h // stride
                ca, cb, cc = next(specs), next(specs), next(specs)
                total += 2 * h * h * ca[1] * ca[0] + 2 * ho * ho * cb[1] * 9 * cb[0] + 2 * ho * ho * cc[1] * cc[0]
                if b == 0:
                    cd = next(specs)
                    total += 2 * ho * ho * cd[1] * cd[0]
                h = ho
        total += 2 * 32 * self.base * 1000
        return total * self.batch

    def setup(self, ctx, dev, rank):
        import torch
        import nm_inputs_cnn
        import paper_2305_14405_b200 as nm
        from paper_2305_14405_b200.harness_cnn import Resnet50Model
        ctx.load_function_table(nm.SLOT_RELU, nm.FUNC_RELU, 2, -8.0, 8.0)
        # the same model on every replica (seed), its own images per rank (seed + rank)
        self.x_np, self.convs, self.fc_w, self.fc_b = nm_inputs_cnn.resnet50_inputs(
            self.batch, seed=self.args.seed, random_bn=True, blocks=self.blocks, base_width=self.base)
        if rank > 0:
            import numpy as np
            import nm_inputs
            rng = np.random.default_rng(self.args.seed + rank)
            self.x_np = nm_inputs.round_to(rng.random(self.x_np.shape, dtype=np.float32), "f16")
        self.model = Resnet50Model(ctx, self.batch, self.convs, self.fc_w, self.fc_b, device=dev, algo=self.args.algo,
                                   blocks=self.blocks, base_width=self.base)
        self.x = torch.from_numpy(self.x_np).to(dev).half()
        self.y = torch.empty((self.batch, 1000), dtype=torch.float16, device=dev)
        self.xh = torch.from_numpy(self.x_np).half().pin_memory()
        self.yh = torch.empty((self.batch, 1000), dtype=torch.float16).pin_memory()
        self.ctx = ctx
        self.h2d = self.batch * 224 * 224 * 3 * 2
        self.d2h = self.batch * 1000 * 2

    def step(self):
        self.model.forward(self.x, self.y)

    def host_step(self):
        m = self.model
        self.ctx.resnet50_forward_host(m.array, m.fc_w, m.fc_b, m.cfg, self.xh, self.yh, self.x, self.y, m.workspace)

    e2e_pipeline = "one stream per step in flight (--streams), each with its own device buffers, workspace and pinned result buffer"

    def host_steps(self, k, stream):
        """k calls of nm_resnet50_forward_host_async, alternating between two streams."""
        m = self.model
        fork_streams(self, stream)
        for i in range(k):
            x, y, ws, yh, st = self.slots[i % len(self.slots)]
            self.ctx.resnet50_forward_host(m.array, m.fc_w, m.fc_b, m.cfg, self.xh, yh, x, y, ws, stream=st, wait=False)
        join_streams(self, stream)

    def device_steps(self, k, stream):
        """k steps on device-resident inputs, alternating between the two streams."""
        m = self.model
        fork_streams(self, stream)
        for i in range(k):
            x, y, ws, yh, st = self.slots[i % len(self.slots)]
            self.ctx.resnet50_forward(m.array, m.fc_w, m.fc_b, m.cfg, x, y, ws, stream=st)
        join_streams(self, stream)

    def _oracle_run(self, n_img):
        import oracle
        import oracle.cnn
        relu = oracle.Table.secant(oracle.RELU, 2, -8.0, 8.0)
        t0 = time.perf_counter()
        oracle.cnn.resnet50(self.x_np[:n_img], self.convs, self.fc_w, self.fc_b, relu, blocks=self.blocks)
        return time.perf_counter() - t0, oracle.num_threads()

    def cpu_baseline(self):
        t1, cores = self._oracle_run(1)
        n = max(1, min(self.batch, int(15.0 / max(t1, 1e-3))))
        secs, cores = self._oracle_run(n)
        return {"value": n / secs, "unit": self.unit, "cores": cores, "kind": "oracle",
                "sample": "%d of %d images through the whole network, %.1f s" % (n, self.batch, secs)}

    def reference_setup(self):
        import nm_inputs_cnn
        self.x_np, self.convs, self.fc_w, self.fc_b = nm_inputs_cnn.resnet50_inputs(1, seed=self.args.seed, random_bn=True)
        self.ref_sample = "1 of %d images through the whole network per step" % self.batch

    def reference_step(self):
        self._oracle_run(1)
        return 1.0


class RowsWorkload:
    """rows: the HBM-bound row kernels on a tensor far larger than L2: PWL LayerNorm over [2^20, 768] bf16
    followed by an element-wise PWL GELU over the result; unit = algorithmic GB (one read and one write
    per element and kernel)."""
    metric = "PWL row kernels GB/s"
    unit = "GB/s"
    dtype = "bf16"
    H = 768

    def __init__(self, args):
        self.args = args
        self.rows = (args.batch or 1024) * 1024
        self.units_per_step = 2 * 2 * self.rows * self.H * 2 / 1e9   # two kernels, read + write, 2 bytes

    def config(self, world):
        return {"workload": "rows_layernorm_gelu_bf16", "rows": self.rows, "hidden": self.H, "pwl_segments": 64,
                "layernorm": "sqrt table then 1/x table" if self.args.ln_two_table else "one rsqrt table",
                "seed": self.args.seed, "parallelism": "replicas" if world > 1 else "single",
                "l2": "each tensor is %.2f GB, far beyond the 126 MB L2; no flush" % (self.rows * self.H * 2 / 1e9)}

    def flops_per_step(self):
        return 0.0

    def _np_inputs(self, rows, seed):
        import nm_inputs
        x = nm_inputs.matrix((rows, self.H), seed, "bf16", 1.0)
        g = nm_inputs.matrix((self.H,), seed + 1, "f32", 0.1) + 1.0
        b = nm_inputs.matrix((self.H,), seed + 2, "f32", 0.1)
        return x, g.astype("float32"), b.astype("float32")

    def setup(self, ctx, dev, rank):
        import torch
        import paper_2305_14405_b200 as nm
        ctx.load_function_table(nm.SLOT_RSQRT, nm.FUNC_RSQRT, 64, 0.05, 8.0)
        ctx.load_function_table(nm.SLOT_GELU, nm.FUNC_GELU, 64, -8.0, 8.0)
        ctx.load_function_table(nm.SLOT_USER0, nm.FUNC_SQRT, 64, 0.05, 8.0)
        ctx.load_function_table(nm.SLOT_USER0 + 1, nm.FUNC_RECIP, 64, 0.2, 3.0)
        self.nm = nm
        # one seeded 2^16-row block, tiled: the kernels' time does not depend on the values
        xb, g, b = self._np_inputs(1 << 16, self.args.seed + rank)
        blk = torch.from_numpy(xb).to(dev).bfloat16()
        self.x = blk.repeat(self.rows // (1 << 16), 1).contiguous()
        self.g = torch.from_numpy(g).to(dev)
        self.b = torch.from_numpy(b).to(dev)
        self.y = torch.empty_like(self.x)
        self.z = torch.empty_like(self.x)
        # end to end on a 2^16-row slice (100 MB each way) so that the default run stays short
        self.e2e_rows = 1 << 16
        self.xh = torch.from_numpy(xb).bfloat16().pin_memory()
        self.zh = torch.empty_like(self.xh).pin_memory()
        self.ctx = ctx
        self.h2d = self.d2h = self.e2e_rows * self.H * 2
        self.e2e_units = 2 * 2 * self.e2e_rows * self.H * 2 / 1e9

    def _ln(self, x, y):
        if self.args.ln_two_table:
            self.ctx.layernorm_pwl_sqrt_recip(x, self.g, self.b, y, self.nm.SLOT_USER0, self.nm.SLOT_USER0 + 1)
        else:
            self.ctx.layernorm_pwl(x, self.g, self.b, y)

    def step(self):
        self._ln(self.x, self.y)
        self.ctx.pwl_apply(self.nm.SLOT_GELU, self.y, self.z)

    def host_step(self):
        import torch
        n = self.e2e_rows
        self.x[:n].copy_(self.xh, non_blocking=True)
        self._ln(self.x[:n], self.y[:n])
        self.ctx.pwl_apply(self.nm.SLOT_GELU, self.y[:n], self.z[:n])
        self.zh.copy_(self.z[:n], non_blocking=True)
        torch.cuda.current_stream().synchronize()

    def roofline(self, prof, peaks, peak_kind):
        out = {}
        for kind in ("layernorm", "pwl_apply"):
            n_k, ms_k, work_k = prof[kind]
            gbs = work_k / (ms_k * 1e-3) / 1e9 if ms_k > 0 else 0.0
            out[kind] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "traffic": None, "avg_launch_us": ms_k / max(n_k, 1) * 1e3,
                         "peak_source": "%s (HBM copy)" % peak_kind}
        main = dict(out["layernorm"], kernel="layernorm")
        return main, {"pwl_apply": out["pwl_apply"]}

    def _oracle_run(self, rows):
        import oracle
        x, g, b = self._np_inputs(rows, self.args.seed)
        t_r = oracle.Table.secant(oracle.RSQRT, 64, 0.05, 8.0)
        t_s = oracle.Table.secant(oracle.SQRT, 64, 0.05, 8.0)
        t_i = oracle.Table.secant(oracle.RECIP, 64, 0.2, 3.0)
        t_g = oracle.Table.secant(oracle.GELU, 64, -8.0, 8.0)
        t0 = time.perf_counter()
        if self.args.ln_two_table:
            y = oracle.layernorm_sqrt_recip(x, g, b, 1e-5, t_s, t_i)
        else:
            y = oracle.layernorm(x, g, b, 1e-5, t_r)
        oracle.pwl_eval(t_g, y)
        return time.perf_counter() - t0, oracle.num_threads()

    def cpu_baseline(self):
        t1, cores = self._oracle_run(1 << 12)
        rows = int(max(1 << 12, min(self.rows, (1 << 12) * 15.0 / max(t1, 1e-4))))
        secs, cores = self._oracle_run(rows)
        return {"value": 2 * 2 * rows * self.H * 2 / 1e9 / secs, "unit": self.unit, "cores": cores, "kind": "oracle",
                "sample": "%d of %d rows through both kernels, %.1f s" % (rows, self.rows, secs)}

    def reference_setup(self):
        self.ref_sample = "%d of %d rows through both kernels per step" % (1 << 14, self.rows)

    def reference_step(self):
        self._oracle_run(1 << 14)
        return 2 * 2 * (1 << 14) * self.H * 2 / 1e9


def make_workload(args):
    if args.workload == "rows":
        return RowsWorkload(args)
    return ResnetWorkload(args) if args.workload == "c5" else EncoderWorkload(args)


def run_reference(args, wl):
    """The CPU oracle, as it stands, on the host cores: each step is a bounded sample of the workload."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    wl.reference_setup()
    for _ in range(args.warmup):
        wl.reference_step()
    t0 = time.perf_counter()
    units = 0.0
    for _ in range(args.steps):
        units += wl.reference_step()
    dt = time.perf_counter() - t0
    value = units / dt
    line = {
        "impl": "reference", "metric": wl.metric, "value": value, "unit": wl.unit, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": wl.config(1),
        "cpu_baseline": {"value": value, "unit": wl.unit, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": wl.ref_sample},
        "e2e": {"value": value, "unit": wl.unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def pick_peak(peaks, clocks, scale=1.0):
    """Which measured bf16 peak a tensor-bound kernel of this run is held against: the burst figure when the
    run kept its clocks (median SM clock within 5 % of the maximum and no power-cap sample while the kernels
    were timed), the sustained figure otherwise.  Returns (peak, name)."""
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    held = bool(mhz and mx and mhz >= 0.95 * mx and "sw_power_cap" not in clocks.get("reasons", []))
    name = "bf16_tflops" if held else "bf16_tflops_sustained"
    return scale * peaks[name], ("burst" if held else "sustained")


def fractions(achieved, peaks, scale=1.0):
    return {"frac_burst": achieved / (scale * peaks["bf16_tflops"]),
            "frac_sustained": achieved / (scale * peaks["bf16_tflops_sustained"]),
            "frac_nominal": achieved / (scale * NOMINAL_BF16_TFLOPS)}


def rows_leg(ctx, nm, dev, peaks, peak_kind, hidden=768, rows=1 << 19, iters=20):
    """The HBM-bound row kernels (PWL LayerNorm, element-wise PWL GELU) on a tensor several times the L2
    (805 MB per tensor at the default size), timed per launch by the library's own events: algorithmic
    bytes (one read and one write per element) / event time, against the measured HBM copy."""
    import torch
    import nm_inputs
    ctx.load_function_table(nm.SLOT_USER0 + 2, nm.FUNC_RSQRT, 64, 0.05, 8.0)
    ctx.load_function_table(nm.SLOT_USER0 + 3, nm.FUNC_GELU, 64, -8.0, 8.0)
    xb = nm_inputs.matrix((1 << 14, hidden), 1234, "bf16", 1.0)
    x = torch.from_numpy(xb).to(dev).bfloat16().repeat(rows // (1 << 14), 1).contiguous()
    g = torch.from_numpy(nm_inputs.matrix((hidden,), 1235, "f32", 0.1) + 1.0).to(dev)
    b = torch.from_numpy(nm_inputs.matrix((hidden,), 1236, "f32", 0.1)).to(dev)
    y = torch.empty_like(x)
    z = torch.empty_like(x)
    for _ in range(3):
        ctx.layernorm_pwl(x, g, b, y, rsqrt_slot=nm.SLOT_USER0 + 2)
        ctx.pwl_apply(nm.SLOT_USER0 + 3, y, z)
    torch.cuda.synchronize()
    ctx.profile_enable(True)
    for _ in range(iters):
        ctx.layernorm_pwl(x, g, b, y, rsqrt_slot=nm.SLOT_USER0 + 2)
        ctx.pwl_apply(nm.SLOT_USER0 + 3, y, z)
    torch.cuda.synchronize()
    prof = ctx.profile_read()
    ctx.profile_enable(False)
    out = {"tensor": "[%d, %d] bf16, %.0f MB per tensor (L2 is 126 MB)" % (rows, hidden, rows * hidden * 2 / 1e6)}
    for kind in ("layernorm", "pwl_apply"):
        n_k, ms_k, work_k = prof[kind]
        gbs = work_k / (ms_k * 1e-3) / 1e9 if ms_k > 0 else 0.0
        out[kind] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": gbs / peaks["hbm_gbs"], "frac_nominal": gbs / NOMINAL_HBM_GBS, "launches": n_k,
                     "avg_launch_us": ms_k / max(n_k, 1) * 1e3, "peak_source": "%s (HBM copy)" % peak_kind}
    del x, y, z
    return out


def other_workload_leg(name, args, dev, steps=10):
    """A short device-resident pass of another workload (its own context, tables and buffers; K steps rotating
    over the streams, CUDA events) so that the default line also carries the int8 encoder's and the CNN's rate."""
    import copy
    import torch
    import paper_2305_14405_b200 as nm
    a = copy.copy(args)
    a.workload, a.hidden, a.layers, a.batch, a.calibrated = name, 0, 0, 0, False
    a.resnet_blocks, a.resnet_width = "", 0
    wl = make_workload(a)
    ctx = nm.Context(torch.cuda.current_device())
    try:
        wl.setup(ctx, dev, 0)
        stream = torch.cuda.current_stream()
        for _ in range(3):
            wl.step()
        many = a.streams >= 2 and hasattr(wl, "device_steps")
        if many:
            wl.device_steps(4, stream)
        torch.cuda.synchronize()
        ctx.check_device_status()
        ctx.launch_count(reset=True)
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        if many:
            wl.device_steps(steps, stream)
        else:
            for _ in range(steps):
                wl.step()
        e1.record(stream)
        torch.cuda.synchronize()
        ctx.check_device_status()
        ms = e0.elapsed_time(e1) / steps
        out = {"workload": wl.config(1)["workload"], "metric": wl.metric, "unit": wl.unit, "dtype": wl.dtype,
               "steps": steps, "streams": a.streams if many else 1, "ms_per_step": ms,
               "value": wl.units_per_step / (ms * 1e-3), "gpu_launches": ctx.launch_count(),
               "whole_step_tflops": wl.flops_per_step() / (ms * 1e-3) / 1e12}
    finally:
        del wl
        ctx.close()
        torch.cuda.empty_cache()
    return out


def main():
    args = parse_args()
    wl = make_workload(args)
    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import torch.distributed as dist
    import paper_2305_14405_b200 as nm

    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    world, rank, local = dist_setup()
    dev = "cuda:%d" % local
    torch.cuda.set_device(local)
    nm.load()
    ctx = nm.Context(local)
    wl.setup(ctx, dev, rank)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        t = torch.tensor([ms], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    warm = max(args.warmup, 3)
    for _ in range(warm):
        wl.step()
    two_streams = args.streams >= 2 and hasattr(wl, "device_steps")
    if two_streams:
        wl.device_steps(4, stream)   # allocates the second slot and warms both streams
        torch.cuda.synchronize()
    ctx.check_device_status()

    # ---- timed region: K steps between two CUDA events on the launching stream, barrier and synchronize
    # on both sides, max over ranks; run `repeats` times, the reported time is the median ----------------
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    time.sleep(0.05)
    reps = []
    launches = 0
    for _ in range(max(1, args.repeats)):
        ev0 = torch.cuda.Event(enable_timing=True)
        ev1 = torch.cuda.Event(enable_timing=True)
        ctx.launch_count(reset=True)
        barrier()
        ev0.record(stream)
        if two_streams:
            wl.device_steps(args.steps, stream)
        else:
            for _ in range(args.steps):
                wl.step()
        ev1.record(stream)
        barrier()
        reps.append(max_over_ranks(ev0.elapsed_time(ev1)) / args.steps)
        launches = ctx.launch_count()
    single_ms = None
    if two_streams:   # the same K steps one after another on one stream, once, for comparison
        barrier()
        ev0.record(stream)
        for _ in range(args.steps):
            wl.step()
        ev1.record(stream)
        barrier()
        single_ms = max_over_ranks(ev0.elapsed_time(ev1)) / args.steps
    sampler.stop()
    ctx.check_device_status()
    srt = sorted(reps)
    ms_step = srt[len(srt) // 2]
    value = world * wl.units_per_step / (ms_step * 1e-3)

    # ---- per-kernel pass: the same steps with every launch bracketed by events, clocks sampled ---------
    per_step = max(1, launches // max(args.steps, 1))
    prof_steps = min(args.steps, max(1, 8000 // per_step))
    prof_sampler = ClockSampler(physical_gpu_index(local))
    prof_sampler.start()
    time.sleep(0.02)
    ctx.profile_enable(True)
    for _ in range(prof_steps):
        wl.step()
    torch.cuda.synchronize()
    prof_sampler.stop()
    prof = ctx.profile_read()
    ctx.profile_enable(False)

    # ---- end to end through the C ABI with host buffers ------------------------------------
    # Every step copies its input from pinned host memory and its result back, inside the timed region.  The
    # encoder and CNN workloads issue the steps through the library's asynchronous host-buffer call on two
    # streams, so that one step's copies overlap the other's kernels (reported under "pipeline"); the same
    # loop with the blocking call, one step at a time, is reported as "serial_ms_per_step".
    e2e_steps = max(4, min(args.steps, 100))   # as many steps as the device-resident region, so that both see the same power state
    wl.host_step()
    barrier()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        wl.host_step()
    e1.record(stream)
    barrier()
    e2e_serial_ms = max_over_ranks(e0.elapsed_time(e1)) / e2e_steps
    e2e_ms = e2e_serial_ms
    if hasattr(wl, "host_steps"):
        wl.host_steps(2, stream)   # allocates the second slot, warms both streams
        barrier()
        e0.record(stream)
        wl.host_steps(e2e_steps, stream)
        e1.record(stream)
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1)) / e2e_steps

    if rank == 0:
        peaks, peak_kind = load_peaks()
        clocks = sampler.summary()
        prof_clocks = prof_sampler.summary()
        total_ms = sum(v[1] for v in prof.values()) or 1.0
        kernels = {k: {"launches_per_step": v[0] / prof_steps, "ms_per_step": v[1] / prof_steps,
                       "share": v[1] / total_ms} for k, v in prof.items() if v[0]}
        gemm_kind = "linear_tc" if prof["linear_tc"][0] else "linear_simt"
        n_l, ms_l, work_l = prof[gemm_kind]
        achieved = work_l / (ms_l * 1e-3) / 1e12 if ms_l > 0 else 0.0
        # int8: the measured bf16 peak times the nominal 2:1 int8:bf16 ratio; fp32 runs on CUDA cores
        scale = {"i8": 2.0, "f32": 0.5}.get(wl.dtype, 1.0)
        peak, which = pick_peak(peaks, prof_clocks, scale)
        roofline = {"bound": "tensor", "kernel": gemm_kind, "achieved": achieved, "peak": peak,
                    "unit": "TFLOP/s", "frac": achieved / peak, "traffic": None,
                    "peak_source": "%s bf16 %s x %.1f: SM clock median %s of %s MHz, reasons %s during the per-kernel pass"
                                   % (peak_kind, which, scale, prof_clocks.get("sm_mhz"), prof_clocks.get("sm_max_mhz"),
                                      prof_clocks.get("reasons")),
                    "avg_launch_us": ms_l / max(n_l, 1) * 1e3, "share_of_step": ms_l / total_ms,
                    "work_per_step": work_l / prof_steps, "ms_per_step": ms_l / prof_steps}
        roofline.update(fractions(achieved, peaks, scale))
        whole = wl.flops_per_step() / (ms_step * 1e-3) / 1e12
        wpeak, wwhich = pick_peak(peaks, clocks, scale)
        whole_step = {"tflops": whole, "peak": wpeak, "frac": whole / wpeak, "peak_source": "%s bf16 %s x %.1f" % (peak_kind, wwhich, scale)}
        whole_step.update(fractions(whole, peaks, scale))
        extra = {}
        for kind in ("layernorm", "quantize", "im2col", "pool"):
            n_k, ms_k, work_k = prof[kind]
            if n_k:
                gbs = work_k / (ms_k * 1e-3) / 1e9
                extra[kind] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                               "frac": gbs / peaks["hbm_gbs"],
                               "note": "in the step (tensors partly L2-resident): algorithmic bytes per launch / event time"}
        for kind in ("attention_tc", "attention_simt"):
            n_a, ms_a, work_a = prof[kind]
            if n_a:
                tf = work_a / (ms_a * 1e-3) / 1e12
                extra[kind] = {"bound": "alu", "achieved_tensor_tflops": tf, "avg_launch_us": ms_a / n_a * 1e3}
        if hasattr(wl, "roofline"):   # a workload whose dominant kernel is not a GEMM brings its own
            roofline, extra = wl.roofline(prof, peaks, peak_kind)
        line = {
            "metric": wl.metric, "value": value, "unit": wl.unit, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": dict(wl.config(world), streams=args.streams if two_streams else 1),
            "streams": {"n": args.streams if two_streams else 1, "single_stream_ms_per_step": single_ms,
                        "note": "the K timed steps rotate over the CUDA streams, each with its own input, "
                                "output and workspace (independent batches in flight together)" if two_streams
                                else "one step after another on one stream"},
            "repeats": {"n": len(reps), "ms_per_step": [round(r, 5) for r in reps], "min": srt[0], "max": srt[-1],
                        "spread": (srt[-1] - srt[0]) / ms_step, "value_is": "median"},
            "clocks": clocks,
            "e2e": {"value": world * getattr(wl, "e2e_units", wl.units_per_step) / (e2e_ms * 1e-3), "unit": wl.unit,
                    "h2d_bytes_per_step": wl.h2d, "d2h_bytes_per_step": wl.d2h, "ms_per_step": e2e_ms,
                    "serial_ms_per_step": e2e_serial_ms,
                    "pipeline": getattr(wl, "e2e_pipeline", "none: one blocking call per step")},
            "gpu_launches": launches,
            "roofline": roofline,
            "roofline_other": extra,
            "kernels": kernels,
            "whole_step": whole_step,
            "whole_step_tflops": whole,
        }
        if isinstance(wl, EncoderWorkload) and not args.no_rows_leg and world == 1:
            try:
                line["roofline_rows"] = rows_leg(ctx, nm, dev, peaks, peak_kind)
            except Exception as e:   # noqa: BLE001 - reported, not hidden
                line["roofline_rows"] = {"error": "%s: %s" % (type(e).__name__, e)}
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = wl.cpu_baseline()
        if (args.workload == "c3" and not args.no_other_legs and world == 1 and not args.hidden and not args.layers):
            legs = []
            for n in ("c4", "c5"):   # a failure here must not cost the main line
                try:
                    legs.append(other_workload_leg(n, args, dev))
                except Exception as e:   # noqa: BLE001 - reported, not hidden
                    legs.append({"workload": n, "error": "%s: %s" % (type(e).__name__, e)})
            line["other_workloads"] = legs
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    ctx.close()


if __name__ == "__main__":
    main()
