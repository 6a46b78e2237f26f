#!/usr/bin/env python
"""Benchmark of the bit-plane mixed-precision convolution path on the five workloads.

The default run (one GPU) times all five configurations in one process and prints ONE JSON line.
The headline (`value`, `ms_per_step`, `roofline`, `e2e`, `cpu_baseline`) is configuration 5, the
largest single-GPU workload: the ImageNet ResNet-50 bottleneck stack at batch 256, 52 convolution
layers chained through fused requantization.  A step is one pass of the whole path over one batch:
ebs_pack_acts at the network entry, one ebs_conv2d_mixed per layer whose epilogue writes the next
layer's packed planes, ebs_dequant of the last layer's accumulators at the exit; weight packing is
done once before timing (it is off the inference path).  `per_config` holds, for each of the five
configurations, the step time, binary and int8 TOPS, the roofline fractions in both output modes
(raw: int32 accumulators + packed planes; fused: packed planes only), cold and warm L2, the literal
AND+POPC path against the POPC pipe, and the CPU oracle timed on a stated sample.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload configN]
"""
from __future__ import annotations

import argparse
import json
import os
import re
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from workloads import gen  # noqa: E402

METRIC = "effective binary TOPS (2*MACs*Wb*Ab per second) of the mixed-precision conv stack"
UNIT = "TOPS"
HEADLINE = "config5"
WORKLOAD_TEXT = {
    "config1": "config1: one 3x3 conv 64->64, 32x32, batch 1, W2A2, seed 0",
    "config2": "config2: ResNet-20 CIFAR-shaped stack, 20 quantized convs, batch 128, (Wb,Ab) in {1..4}^2, seed 0",
    "config3": "config3: ResNet-18 ImageNet-shaped quantized convs, batch 64, (Wb,Ab) in {2..6}^2, seed 0",
    "config4": "config4: 4096^3 bit-plane GEMM as a 1x1 convolution over 64x64 pixels, all 64 (Wb,Ab) pairs, seed 0",
    "config5": "config5: ResNet-50 ImageNet-shaped bottleneck stack, 52 convs, batch 256, (Wb,Ab) in {2..8}^2, seed 0, "
               "chained through fused requantization",
}
SM_COUNT, POPC_LANES_PER_CLK_SM = 148, 16
TRAFFIC_PROFILE = os.path.join(ROOT, "profiles", "conv_dram_traffic.md")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "sm_max_mhz": 1965.0}, "fallback"


def int8_tensor_peak_tops(peaks: dict) -> float:
    """Dense int8 tensor peak in TOPS: the measured bf16 burst figure times the nominal int8:bf16 ratio (2)."""
    return 2.0 * float(peaks.get("bf16_tflops", 1590.0))


def popc_pipe_peak_tops(sm_max_mhz: float) -> float:
    """Binary TOPS of the POPC pipe: 16 lanes/clk/SM x 32 bit x 148 SMs x clock, 2 ops per bit pair."""
    return 2.0 * SM_COUNT * POPC_LANES_PER_CLK_SM * 32 * sm_max_mhz * 1e6 / 1e12


def ncu_traffic_per_launch(workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per conv launch for a workload, from the committed ncu summary
    (a line `traffic_bytes_per_launch[<workload>] = <integer>`); None if the summary has no such line."""
    try:
        with open(TRAFFIC_PROFILE) as f:
            m = re.search(r"traffic_bytes_per_launch\[%s\]\s*=\s*(\d+)" % re.escape(workload), f.read())
        return int(m.group(1)) if m else None
    except OSError:
        return None


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.index, self.period, self.samples, self.reasons, self.max_mhz = index, period_s, [], set(), None
        self._stop_evt = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
                mask = get(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---------------------------------------------------------------------------- workloads (layer lists, wiring)

def workload_specs(name: str):
    """(specs, chained) of a configuration; chained: layer l+1 reads layer l's packed output."""
    if name == "config1":
        return gen.config1(0), False
    if name == "config2":
        return [s for s in gen.config2(0) if s.layer.quantized], False
    if name == "config3":
        return gen.config3(0), False
    if name == "config4":
        return [gen.config4(wb, ab) for wb in range(1, 9) for ab in range(1, 9)], False
    if name == "config5":
        return gen.config5(0), True
    raise KeyError(name)


def consumer_bits(specs, i, chained):
    """Activation bitwidth the output of layer i is requantized to: that of the layer that reads it."""
    if not chained:
        return specs[(i + 1) % len(specs)].a_bits
    j = i + 1
    while j < len(specs) and specs[j].layer.role == "shortcut":
        j += 1
    return specs[j].a_bits if j < len(specs) else specs[i].a_bits


# ---------------------------------------------------------------------------- GPU arm

class Layer:
    """Device buffers and descriptors of one layer (plumbing only)."""

    def __init__(self, ebs, spec, next_bits, dev, px=None, qa=None, qw_dev=None, pw=None, want_host=False):
        L = spec.layer
        self.spec, self.n, self.next_bits = spec, spec.batch, next_bits
        self.d = ebs.conv_desc(L.c_in, L.c_out, L.k, L.k, L.stride, L.stride, L.pad, L.pad, spec.w_bits, spec.a_bits,
                               spec.w_scale, spec.a_scale)
        self.x = self.x_host = None
        self.px_bytes = ebs.ebs_packed_act_bytes(self.n, L.h_in, L.w_in, L.c_in, spec.a_bits)
        if px is None:                                              # an input of its own: generator codes, packed here
            qa = gen.act_codes(spec).astype(np.uint8) if qa is None else qa
            xh = torch.from_numpy(np.ascontiguousarray(qa.transpose(0, 2, 3, 1)))    # NHWC codes
            self.x_host = xh.pin_memory() if want_host else xh
            self.x = self.x_host.to(dev)
            px = torch.empty(self.px_bytes // 4, dtype=torch.int32, device=dev)
        self.px = px
        if pw is None:
            qw_dev = torch.from_numpy(gen.weight_codes(spec).astype(np.int8)).to(dev) if qw_dev is None else qw_dev
            pw = torch.empty(ebs.ebs_packed_weight_bytes(self.d) // 4, dtype=torch.int32, device=dev)
            ebs.ebs_pack_weights(qw_dev, ebs.EBS_I8_CODES, ebs.EBS_NCHW, self.d, pw)
        self.pw = pw
        ho, wo = L.h_out, L.w_out
        self.pixels = self.n * ho * wo
        self.outputs = self.pixels * L.c_out
        self.acc = None                                             # allocated by want_acc()
        self.pn_bytes = ebs.ebs_packed_act_bytes(self.n, ho, wo, L.c_out, next_bits)
        self.pn = torch.empty(self.pn_bytes // 4, dtype=torch.int32, device=dev)
        self.next_scale = 4.0 * spec.w_scale * spec.a_scale * L.c_in
        self.epi = ebs.epilogue(relu=True, next_a_bits=next_bits, next_a_scale=self.next_scale)
        self.S = float(np.float32(spec.w_scale) * np.float32(spec.a_scale))
        self.ops = gen.binary_ops(spec)
        self.int8_ops = self.ops // (spec.w_bits * spec.a_bits)    # 2 * MACs
        co16 = (L.c_out + 15) // 16 * 16
        self.w_plane_bytes = ebs.ebs_packed_weight_plane_bytes(self.d)
        self.w_image_bytes = L.k * L.k * ((L.c_in + 31) // 32) * co16 * 32
        self.dev = dev

    def want_acc(self):
        if self.acc is None:
            L = self.spec.layer
            self.acc = torch.empty((self.n, L.h_out, L.w_out, L.c_out), dtype=torch.int32, device=self.dev)
        return self.acc

    def set_step(self, ebs, step: float):
        self.next_scale = float(step)
        self.epi = ebs.epilogue(relu=True, next_a_bits=self.next_bits, next_a_scale=self.next_scale)

    def run_pack(self, ebs):
        L = self.spec.layer
        ebs.ebs_pack_acts(self.x, ebs.EBS_U8_CODES, ebs.EBS_NHWC, self.n, L.c_in, L.h_in, L.w_in, self.spec.a_bits,
                          self.spec.a_scale, self.px)

    def run_conv(self, ebs, raw: bool, variant=-1):
        L = self.spec.layer
        ebs.ebs_conv2d_mixed(self.px, self.n, L.h_in, L.w_in, self.pw, self.d, self.epi, self.want_acc() if raw else None,
                             None, self.pn, variant=variant)

    def bytes_alg(self, raw: bool, literal: bool = False):
        """Algorithmic bytes of one launch: packed input planes + weights as the kernel family reads them (bit planes for
        the integer-pipe kernels, the byte image for the tensor-pipe kernels) + packed output planes (+ int32
        accumulators in raw mode)."""
        w = self.w_plane_bytes if literal else self.w_image_bytes
        return self.px_bytes + w + self.pn_bytes + (4 * self.outputs if raw else 0)


def dist_setup(n_gpus: int):
    """One process per GPU under torchrun; returns (rank, world, local_rank)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        if not dist.is_initialized():
            dist.init_process_group(backend=backend)
        return dist.get_rank(), world, int(os.environ.get("LOCAL_RANK", "0"))
    return 0, 1, 0


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of a scalar (the only collective: the data path itself shards with none)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


# ---------------------------------------------------------------------------- CPU oracle arm

ORACLE_SAMPLES = {
    # workload: (what one pass runs, how it scales to the full workload)
    "config1": "the layer at full size (batch 1)",
    "config2": "all 20 quantized layers at batch {b} of 128",
    "config3": "all 19 layers at batch {b} of 64 (scaled from subset)",
    "config4": "the W4A4 GEMM on {b} of 4096 rows (scaled from subset; the integer oracle's time does not depend on the bitwidths)",
    "config5": "all 52 layers at batch {b} of 256, each on generator codes (scaled from subset)",
}


class OracleWorkload:
    """The CPU oracle on a bounded sample of a workload; codes are generated outside the timing."""

    def __init__(self, workload: str, batch: int):
        import oracle
        oracle.build()
        self.oracle, self.workload, self.batch = oracle, workload, batch
        if workload == "config4":
            spec = gen.config4(4, 4)
            rows = batch                                       # `batch` counts GEMM rows here: 1 x rows pixels
            qa = gen.act_codes(spec)[:, :, :1, :rows]
            self.specs, self.data = [spec], [(np.ascontiguousarray(qa), gen.weight_codes(spec))]
            self.ops = 2 * rows * spec.layer.c_in * spec.layer.c_out * 16
            self.next_bits = [4]
        else:
            self.specs, chained = workload_specs(workload)
            b = min(batch, self.specs[0].batch)
            self.batch = b
            self.data = [(gen.act_codes(s, batch=b), gen.weight_codes(s)) for s in self.specs]
            self.ops = sum(gen.binary_ops(s, batch=b) for s in self.specs)
            self.next_bits = [consumer_bits(self.specs, i, chained) for i in range(len(self.specs))]

    def step(self) -> float:
        t0 = time.perf_counter()
        for s, (qa, qw), nb in zip(self.specs, self.data, self.next_bits):
            L = s.layer
            acc = self.oracle.conv2d_codes(qa, qw, (L.stride, L.stride), (L.pad, L.pad))
            step = np.float32(4.0 * s.w_scale * s.a_scale * L.c_in)
            self.oracle.epilogue(acc, self.oracle.combined_scale(s.w_scale, s.a_scale), relu=True, next_bits=nb,
                                 inv_next=np.float32(1.0) / step)
        return time.perf_counter() - t0

    def describe(self) -> str:
        return ORACLE_SAMPLES[self.workload].format(b=self.batch)


def oracle_sample_size(workload: str, budget_s: float, n_steps: int) -> int:
    """Largest sample (images, or GEMM rows for config4) for which n_steps oracle passes fit the time budget."""
    if workload == "config1":
        return 1
    # upper limits keep the generation of the sample's codes (host, untimed) and the run within minutes
    full = {"config2": 128, "config3": 8, "config4": 256, "config5": 4}[workload]
    small = {"config2": 2, "config3": 1, "config4": 16, "config5": 1}[workload]
    probe = OracleWorkload(workload, small)
    probe.step()
    per_unit = probe.step() / small
    return int(max(small, min(full, budget_s / max(n_steps, 1) / per_unit)))


def cpu_baseline_sample(workload: str, budget_s: float):
    """The oracle, as it stands, timed on this host's cores on a bounded sample (a reported baseline)."""
    wl = OracleWorkload(workload, oracle_sample_size(workload, budget_s, 3))
    wl.step()
    reps = 20 if workload == "config1" else 2
    times = [wl.step() for _ in range(reps)]
    dt = float(np.mean(times))
    return {"value": wl.ops / dt / 1e12, "unit": UNIT, "cores": wl.oracle.num_threads(), "kind": "oracle",
            "sample": f"{wl.describe()}: direct integer conv + fp32 epilogue with requantization, "
                      f"mean of {reps} passes of {dt:.3f} s"}


def run_reference(args):
    rank, world, _ = dist_setup(args.gpus)
    if rank != 0:
        return
    workload = HEADLINE if args.workload == "all" else args.workload
    wl = OracleWorkload(workload, oracle_sample_size(workload, 120.0, args.steps + args.warmup))
    for _ in range(args.warmup):
        wl.step()
    times = [wl.step() for _ in range(args.steps)]
    dt = float(np.mean(times))
    value = wl.ops / dt / 1e12
    base = {"value": value, "unit": UNIT, "cores": wl.oracle.num_threads(), "kind": "oracle",
            "sample": f"each step: {wl.describe()}"}
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[workload], "sample": wl.describe()},
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ---------------------------------------------------------------------------- measurement helpers

class Timer:
    def __init__(self, stream, flush):
        self.stream, self.flush = stream, flush

    def graph_ms(self, graph, reps: int, cold: bool) -> float:
        """Mean CUDA-event time of one replay; cold = the 256 MB flush buffer is rewritten before every replay."""
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        if not cold:
            graph.replay()
        for e0, e1 in ev:
            if cold:
                self.flush.zero_()
            e0.record(self.stream)
            graph.replay()
            e1.record(self.stream)
        torch.cuda.synchronize()
        return float(np.mean([e0.elapsed_time(e1) for e0, e1 in ev]))


def capture(fn):
    """Records fn's launches into a CUDA graph so that replay is not bound by host launch overhead."""
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        fn()                                                    # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    with torch.cuda.graph(g):
        fn()
    return g


def build_layers(ebs, name, dev, want_host=False):
    """Layers of a workload with their device buffers; chained workloads share buffers along the chain."""
    specs, chained = workload_specs(name)
    layers = []
    if name == "config4":
        # one activation tensor per Ab and one weight tensor per Wb serve the 64 pairs
        acts, wts = {}, {}
        for ab in range(1, 9):
            s = gen.config4(1, ab)
            first = Layer(ebs, s, ab, dev)
            first.run_pack(ebs)
            acts[ab] = first.px
        for wb in range(1, 9):
            wts[wb] = torch.from_numpy(gen.weight_codes(gen.config4(wb, 1)).astype(np.int8)).to(dev)
        for i, s in enumerate(specs):
            layers.append(Layer(ebs, s, s.a_bits, dev, px=acts[s.a_bits], qw_dev=wts[s.w_bits]))
        torch.cuda.synchronize()
        return specs, layers, chained
    block_in = None
    for i, s in enumerate(specs):
        nb = consumer_bits(specs, i, chained)
        if not chained or i == 0:
            L = Layer(ebs, s, nb, dev, want_host=want_host)
            L.run_pack(ebs)
        else:
            prev = next(p for p in reversed(layers) if p.spec.layer.role != "shortcut")
            src = block_in if s.layer.role == "shortcut" else prev.pn
            L = Layer(ebs, s, nb, dev, px=src)
        if chained and s.layer.name.endswith("c1"):
            block_in = L.px
        layers.append(L)
    torch.cuda.synchronize()
    return specs, layers, chained


def calibrate_chain(ebs, layers):
    """Requantization steps of a chained stack, fixed once before timing (set-up, untimed): each layer's step maps
    the 99.5th percentile of its ReLU output (sampled) onto the top code, so that the codes handed down the chain
    use their whole range.  torch is used for the percentile only."""
    for L in layers:
        lay = L.spec.layer
        y = torch.empty((L.n, lay.h_out, lay.w_out, lay.c_out), dtype=torch.float32, device=L.dev)
        epi = ebs.epilogue(relu=True)
        ebs.ebs_conv2d_mixed(L.px, L.n, lay.h_in, lay.w_in, L.pw, L.d, epi, None, y, None)
        flat = y.flatten()
        sample = flat[:: max(1, flat.numel() // (1 << 20))].float()
        top = float(torch.quantile(sample, 0.995).item())
        L.set_step(ebs, max(top, 1e-6) / ((1 << L.next_bits) - 1))
        del y, flat, sample
        L.run_conv(ebs, raw=False)                              # the next layer calibrates on this output
    torch.cuda.synchronize()


def layer_roofs(L: Layer, raw: bool, peak_tops: float, hbm_gbs: float):
    t_tensor = L.int8_ops / (peak_tops * 1e12)
    t_hbm = L.bytes_alg(raw) / (hbm_gbs * 1e9)
    return t_tensor, t_hbm


def measure_config(ebs, name, dev, timer, peaks, args, sm_max, detail: bool):
    """All numbers of one configuration (see the module docstring)."""
    peak_tops, hbm_gbs = int8_tensor_peak_tops(peaks), float(peaks.get("hbm_gbs", 6650.0))
    specs, layers, chained = build_layers(ebs, name, dev)
    if chained:
        calibrate_chain(ebs, layers)
    step_raw = not chained                       # the chained stack hands packed planes down; the others also keep int32 results
    total_ops = sum(L.ops for L in layers)
    total_int8 = sum(L.int8_ops for L in layers)
    n_img = specs[0].batch
    last = layers[-1]
    y_exit = torch.empty((last.pixels, last.spec.layer.c_out), dtype=torch.float32, device=dev)

    def one_step():
        layers[0].run_pack(ebs) if layers[0].x is not None else None
        for L in layers[:-1]:
            L.run_conv(ebs, raw=step_raw)
        last.run_conv(ebs, raw=True)                            # the exit layer's accumulators feed ebs_dequant
        ebs.ebs_dequant(last.want_acc(), last.pixels, last.spec.layer.c_out, last.S, None, None, True, y_exit)

    launches_per_step = len(layers) + 1 + (1 if layers[0].x is not None else 0)
    reps_inner = 1000 if name == "config1" else 1              # a one-layer step is timed as 1000 back-to-back launches
    step_graph = capture(lambda: [one_step() for _ in range(reps_inner)])
    reps = max(3, min(args.steps, 20))
    out = {"workload": WORKLOAD_TEXT[name], "layers": len(layers), "batch": n_img,
           "step": ("pack at the entry, %d fused conv launches (%s), dequant at the exit"
                    % (len(layers), "int32 accumulators + packed planes" if step_raw else "packed planes only, chained")),
           "launches_per_step": launches_per_step}
    if name == "config1":
        out["step"] += "; timed as 1000 back-to-back steps in one graph, per-step time reported"
    step_ms = timer.graph_ms(step_graph, reps, cold=True) / reps_inner
    out["ms_per_step"] = step_ms
    out["binary_tops"] = total_ops / (step_ms * 1e-3) / 1e12
    out["int8_tops"] = total_int8 / (step_ms * 1e-3) / 1e12
    out["imgs_per_s"] = n_img / (step_ms * 1e-3)
    if args.step_only:
        return out, layers, step_graph, one_step, launches_per_step, total_ops, total_int8

    # the conv launches alone, both output modes, cold (flush before every replay) and warm (replays back to back)
    modes = {}
    per_layer = {}
    for mode, raw in (("raw", True), ("fused", False)):
        g = capture(lambda raw=raw: [[L.run_conv(ebs, raw=raw) for L in layers] for _ in range(reps_inner)])
        cold = timer.graph_ms(g, reps, cold=True) / reps_inner
        warm = timer.graph_ms(g, reps, cold=False) / reps_inner
        del g
        # per-layer times: each layer's launch 10 times back to back in a graph (L2-warm)
        lay_ms = np.zeros(len(layers))
        for i, L in enumerate(layers):
            gl = capture(lambda L=L, raw=raw: [L.run_conv(ebs, raw=raw) for _ in range(10)])
            lay_ms[i] = timer.graph_ms(gl, 2, cold=False) / 10.0
            del gl
        roofs = [layer_roofs(L, raw, peak_tops, hbm_gbs) for L in layers]
        roof_s = np.array([max(r) for r in roofs])
        sum_tensor, sum_hbm = sum(r[0] for r in roofs), sum(r[1] for r in roofs)
        fr = roof_s * 1e3 / lay_ms
        bytes_alg = sum(L.bytes_alg(raw) for L in layers)
        modes[mode] = {
            "outputs": "int32 accumulators + packed planes" if raw else "packed planes only",
            "conv_ms_cold": cold, "conv_ms_warm": warm, "sum_layer_ms_warm": float(lay_ms.sum()),
            "sum_layer_roofs_ms": float(roof_s.sum() * 1e3),
            "bound": "tensor" if sum_tensor >= sum_hbm else "hbm",
            "sum_tensor_roofs_ms": sum_tensor * 1e3, "sum_hbm_roofs_ms": sum_hbm * 1e3,
            "frac_cold": float(roof_s.sum() * 1e3 / cold), "frac_warm": float(roof_s.sum() * 1e3 / warm),
            "frac_of_layer_roofs": float(roof_s.sum() * 1e3 / lay_ms.sum()),
            "layer_frac_min": float(fr.min()), "layer_frac_max": float(fr.max()),
            "layers_at_or_above_half": int((fr >= 0.5).sum()),
            "algorithmic_bytes": int(bytes_alg), "gbs_cold": bytes_alg / (cold * 1e-3) / 1e9,
            "int8_tops_cold": total_int8 / (cold * 1e-3) / 1e12, "binary_tops_cold": total_ops / (cold * 1e-3) / 1e12,
        }
        per_layer[mode] = [
            {"name": L.spec.layer.name, "wb": L.spec.w_bits, "ab": L.spec.a_bits, "us": round(float(t) * 1e3, 2),
             "tops": round(L.ops / (t * 1e-3) / 1e12, 1), "int8_tops": round(L.int8_ops / (t * 1e-3) / 1e12, 1),
             "bytes": int(L.bytes_alg(raw)), "roof_us": round(float(r) * 1e6, 2),
             "roof": "tensor" if rr[0] >= rr[1] else "hbm", "frac_of_roof": round(float(f), 3)}
            for L, t, r, rr, f in zip(layers, lay_ms, roof_s, roofs, fr)]
    out["modes"] = modes
    if detail or name in ("config1", "config4"):
        out["per_layer"] = per_layer
    else:
        out["per_layer"] = {m: [{k: pl[k] for k in ("name", "wb", "ab", "us", "frac_of_roof")} for pl in v]
                            for m, v in per_layer.items()}

    # context (not the paper's method): the same layers with the activations as unpacked u8 codes, which skips the
    # bit-plane expansion at 8 / Ab times the activation traffic; packed output only; layers it cannot run are skipped
    ctx_ms, ctx_ref_ms, ctx_layers = 0.0, 0.0, 0
    for i, L in enumerate(layers):
        lay = L.spec.layer
        if lay.c_in % 32 != 0:
            continue
        xb = torch.randint(0, 1 << L.spec.a_bits, (L.n, lay.h_in, lay.w_in, lay.c_in), dtype=torch.uint8, device=dev)
        try:
            gl = capture(lambda L=L, lay=lay, xb=xb: [ebs.ebs_conv2d_i8(xb, L.n, lay.h_in, lay.w_in, L.pw, L.d, L.epi, None, None, L.pn)
                                                     for _ in range(10)])
        except ebs.EbsError:
            del xb
            continue
        ctx_ms += timer.graph_ms(gl, 2, cold=False) / 10.0
        ctx_ref_ms += float(per_layer["fused"][i]["us"]) * 1e-3
        ctx_layers += 1
        del gl, xb
    out["i8_context_path"] = {
        "what": "ebs_conv2d_i8: activations as unpacked u8 NHWC codes instead of bit planes (context, not the paper's method)",
        "layers": ctx_layers, "sum_layer_ms_warm": ctx_ms, "bit_plane_path_same_layers_ms": ctx_ref_ms,
        "bit_plane_over_i8": (ctx_ref_ms / ctx_ms) if ctx_ms > 0 else None}

    # the same conv launches on the integer-pipe kernels only: the plane-pair double sum evaluated literally
    # (AND + POPC + shift-add per plane pair), held against the POPC pipe's peak
    lit_graph = capture(lambda: [L.run_conv(ebs, raw=True, variant=-2) for L in layers])
    lit_reps = 1 if name in ("config4", "config5") else 3
    lit_ms = timer.graph_ms(lit_graph, lit_reps, cold=True)
    del lit_graph
    popc_peak = popc_pipe_peak_tops(sm_max)
    out["literal_bitplane_path"] = {
        "kernel": "conv_popc_kernel (variant -2: the library's choice among the integer-pipe kernels), raw outputs",
        "conv_ms": lit_ms, "binary_tops": total_ops / (lit_ms * 1e-3) / 1e12, "popc_pipe_peak_tops": popc_peak,
        "frac_of_popc_pipe": total_ops / (lit_ms * 1e-3) / 1e12 / popc_peak}
    return out, layers, step_graph, one_step, launches_per_step, total_ops, total_int8


def streaming_leg(ebs, dev, stream, hbm_gbs):
    """The streaming kernels (rows a2 and a6, search-stage forward): achieved GB/s of algorithmic bytes.  Every kernel
    reads more than the 126 MB of L2 per launch (fp32 tensors: 51 M values = 205 MB; the u8 code tensor has four times
    the pixels for that), so consecutive launches find nothing of their input in cache; each measurement is a CUDA graph
    of five back-to-back launches, so that the host's launch cost (about 15 us per call through ctypes, as long as some of
    these kernels run) is not in the figure."""
    sn, sh, sc, sab = 256, 56, 64, 4                                   # ResNet-50 layer-1 activations: 51 M values
    vals = sn * sh * sh * sc
    un = 4 * sn                                                        # images of the u8 tensor (205 MB)
    xf = torch.rand((sn, sh, sh, sc), dtype=torch.float32, device=dev)
    xu = torch.randint(0, 16, (un, sh, sh, sc), dtype=torch.uint8, device=dev)
    pk = torch.empty(ebs.ebs_packed_act_bytes(un, sh, sh, sc, sab) // 4, dtype=torch.int32, device=dev)
    ai = torch.randint(-1000, 1000, (sn * sh * sh, sc), dtype=torch.int32, device=dev)
    yo = torch.empty((sn * sh * sh, sc), dtype=torch.float32, device=dev)

    def gbs(fn, nbytes, reps=3, inner=5):
        g = capture(lambda: [fn() for _ in range(inner)])
        g.replay()
        tot = 0.0
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            g.replay()
            b.record(stream)
            torch.cuda.synchronize()
            tot += a.elapsed_time(b)
        del g
        return nbytes / (tot / (reps * inner) * 1e-3) / 1e9

    out_b = vals * sab // 8
    res = {
        "tensor": f"{sn}x{sh}x{sh}x{sc} NHWC fp32 / int32 ({un} images for u8 codes), {sab} planes", "hbm_peak_gbs": hbm_gbs,
        "timing": "CUDA graph of 5 back-to-back launches, inputs larger than L2",
        "pack_acts_fp32_gbs": gbs(lambda: ebs.ebs_pack_acts(xf, ebs.EBS_F32, ebs.EBS_NHWC, sn, sc, sh, sh, sab, 0.07, pk),
                                  vals * 4 + out_b),
        "pack_acts_u8_gbs": gbs(lambda: ebs.ebs_pack_acts(xu, ebs.EBS_U8_CODES, ebs.EBS_NHWC, un, sc, sh, sh, sab, 1.0, pk),
                                4 * (vals + out_b)),
        "pack_acts_fp32_nchw_gbs": gbs(lambda: ebs.ebs_pack_acts(xf, ebs.EBS_F32, ebs.EBS_NCHW, sn, sc, sh, sh, sab, 0.07, pk),
                                       vals * 4 + out_b),
        "dequant_gbs": gbs(lambda: ebs.ebs_dequant(ai, sn * sh * sh, sc, 0.01, None, None, True, yo), vals * 8),
    }
    # search-stage forward (Eq. 6-7), five candidate bitwidths: 4 B in + 4 B out per value; the weight form
    # reads the tensor once more for max|w|
    cand_bits, cand_coeff = [1, 2, 3, 4, 5], [0.1, 0.15, 0.4, 0.25, 0.1]
    scratch = torch.zeros(4, dtype=torch.int32, device=dev)
    xo = torch.empty_like(xf)
    res["search_act_forward_gbs"] = gbs(lambda: ebs.ebs_search_act_forward(xf, 6.0, cand_bits, cand_coeff, xo), vals * 8)
    res["search_weight_forward_gbs"] = gbs(
        lambda: ebs.ebs_search_weight_forward(xf, cand_bits, cand_coeff, xo, scratch), vals * 12)
    return res


def network_leg(ebs, dev, stream, flush, reps):
    """ResNet-20 forward passes per second at batch 128 through paper_2003_07577_b200.network."""
    from paper_2003_07577_b200.network import BasicBlockNet, FusedBasicBlockNet, calibrated_plans
    from types import SimpleNamespace
    specs = gen.resnet20_network(0, 128)
    n = specs[0].batch
    imgs_host = torch.from_numpy(np.ascontiguousarray(gen.images_u8(0, n).astype(np.uint8).transpose(0, 2, 3, 1))).pin_memory()
    imgs = imgs_host.to(dev)
    recs = [SimpleNamespace(name=s.layer.name, role=s.layer.role, c_in=s.layer.c_in, c_out=s.layer.c_out, k=s.layer.k,
                            stride=s.layer.stride, pad=s.layer.pad, h_in=s.layer.h_in, w_in=s.layer.w_in,
                            w_bits=s.w_bits, a_bits=s.a_bits, w_scale=s.w_scale) for s in specs]
    wts = {s.layer.name: torch.from_numpy(gen.weight_codes(s).astype(np.int8)).to(dev) for s in specs}
    plans = calibrated_plans(recs, wts, imgs, dev)
    net = BasicBlockNet(plans, dev)
    fused = FusedBasicBlockNet(plans, dev)              # the same network as one launch, activations resident on chip
    out = {}
    g = capture(lambda: out.__setitem__("logits", net.forward(imgs)))
    ms = []
    for _ in range(reps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        g.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    logits_host = torch.empty((n, specs[-1].layer.c_out), dtype=torch.float32).pin_memory()
    t0 = time.perf_counter()
    for _ in range(reps):
        imgs.copy_(imgs_host, non_blocking=True)
        g.replay()
        logits_host.copy_(out["logits"], non_blocking=True)
        torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / reps
    # the whole-network kernel: one launch per batch (no graph needed), cold L2
    fused_logits = fused.forward(imgs)
    torch.cuda.synchronize()
    same = bool((fused_logits == out["logits"]).all().item())
    fms = []
    for _ in range(reps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        fused.forward(imgs)
        e1.record(stream)
        torch.cuda.synchronize()
        fms.append(e0.elapsed_time(e1))
    t0 = time.perf_counter()
    for _ in range(reps):
        imgs.copy_(imgs_host, non_blocking=True)
        lg = fused.forward(imgs)
        logits_host.copy_(lg, non_blocking=True)
        torch.cuda.synchronize()
    fused_e2e_s = (time.perf_counter() - t0) / reps
    ft = float(np.mean(fms)) * 1e-3
    ops = sum(gen.binary_ops(s) for s in specs)
    t = float(np.mean(ms)) * 1e-3
    return {"model": "ResNet-20 (CIFAR), basic blocks with fused shortcuts, average pool, classifier", "batch": n,
            "ms_per_batch": t * 1e3, "imgs_per_s": n / t, "effective_tops": ops / t / 1e12,
            "launches_per_batch": net.launches_per_forward, "l2": "cold (flushed before every replay)",
            "e2e_imgs_per_s": n / e2e_s, "e2e_note": "pinned host images in, host logits out, wall clock",
            "fused": {"kernel": "fused_resnet_kernel: one launch, one thread block per image, activation bytes resident "
                                "in shared memory", "ms_per_batch": ft * 1e3, "imgs_per_s": n / ft,
                      "effective_tops": ops / ft / 1e12, "e2e_imgs_per_s": n / fused_e2e_s,
                      "logits_identical_to_layerwise": same},
            "finite_logits": bool(torch.isfinite(out["logits"]).all().item())}


def resnet18_leg(ebs, dev, stream, flush, reps, batch=64):
    """ImageNet ResNet-18 forward passes per second (224x224 images) through paper_2003_07577_b200.network: 7x7 first
    convolution at 8 bits, max pooling on packed codes, basic blocks with fused shortcuts, average pooling, classifier."""
    from paper_2003_07577_b200.network import BasicBlockNet, calibrated_plans
    from types import SimpleNamespace
    specs = gen.resnet18_network(0, batch)
    imgs_host = torch.from_numpy(np.ascontiguousarray(gen.images_u8(0, batch, 224, 224).astype(np.uint8).transpose(0, 2, 3, 1))).pin_memory()
    imgs = imgs_host.to(dev)
    recs = [SimpleNamespace(name=s.layer.name, role=s.layer.role, c_in=s.layer.c_in, c_out=s.layer.c_out, k=s.layer.k,
                            stride=s.layer.stride, pad=s.layer.pad, h_in=s.layer.h_in, w_in=s.layer.w_in,
                            w_bits=s.w_bits, a_bits=s.a_bits, w_scale=s.w_scale) for s in specs]
    wts = {s.layer.name: torch.from_numpy(gen.weight_codes(s).astype(np.int8)).to(dev) for s in specs}
    pool = (3, 2, 1)
    net = BasicBlockNet(calibrated_plans(recs, wts, imgs, dev, pool=pool), dev, pool=pool)
    out = {}
    g = capture(lambda: out.__setitem__("logits", net.forward(imgs)))
    ms = []
    for _ in range(reps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        g.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    logits_host = torch.empty((batch, specs[-1].layer.c_out), dtype=torch.float32).pin_memory()
    t0 = time.perf_counter()
    for _ in range(reps):
        imgs.copy_(imgs_host, non_blocking=True)
        g.replay()
        logits_host.copy_(out["logits"], non_blocking=True)
        torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / reps
    t = float(np.mean(ms)) * 1e-3
    ops = sum(gen.binary_ops(s) for s in specs)
    return {"model": "ResNet-18 (ImageNet, 224x224): 7x7 first convolution at W8A8, 3x3/2 max pooling on packed codes, basic "
                     "blocks with fused shortcuts, average pool, classifier", "batch": batch, "ms_per_batch": t * 1e3,
            "imgs_per_s": batch / t, "effective_tops": ops / t / 1e12, "launches_per_batch": net.launches_per_forward,
            "l2": "cold (flushed before every replay)", "e2e_imgs_per_s": batch / e2e_s,
            "finite_logits": bool(torch.isfinite(out["logits"]).all().item())}


def run_gpu(args):
    from paper_2003_07577_b200 import binding as ebs
    ebs.lib()
    rank, world, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    peaks, peak_kind = measured_peaks()
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > 126 MB L2
    timer = Timer(stream, flush)
    sm_max = float(peaks.get("sm_max_mhz", 1965.0))
    headline = HEADLINE if args.workload == "all" else args.workload
    others = [c for c in ("config1", "config2", "config3", "config4") if c != headline] \
        if (args.workload == "all" and world == 1) else []

    # ---- the other configurations first (their buffers are released before the headline workload is built)
    per_config = {}
    for name in others:
        res, layers, g, _, _, _, _ = measure_config(ebs, name, dev, timer, peaks, args, sm_max, detail=False)
        if not args.no_cpu_baseline:
            res["cpu_baseline"] = cpu_baseline_sample(name, 4.0)
        per_config[name] = res
        del layers, g
        torch.cuda.empty_cache()

    # ---- the headline configuration: the timed steps of the contract
    res, layers, step_graph, one_step, launches_per_step, total_ops, total_int8 = measure_config(
        ebs, headline, dev, timer, peaks, args, sm_max, detail=True)
    chained = headline == "config5"
    inner = 1000 if headline == "config1" else 1
    for _ in range(max(args.warmup, 3)):
        step_graph.replay()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    torch.cuda.synchronize()
    sampler.start()
    wall0 = time.perf_counter()
    for e0, e1 in ev:
        flush.zero_()                                               # cold L2 for every timed step
        e0.record(stream)
        step_graph.replay()
        e1.record(stream)
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    barrier()
    total_ms = max_over_ranks(float(sum(e0.elapsed_time(e1) for e0, e1 in ev)), dev)
    ms_per_step = total_ms / args.steps / inner
    if args.step_only:
        # the short form for profiler captures: the timed steps alone, none of the per-layer, per-mode or context legs
        sampler.stop()
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": world * total_ops / (ms_per_step * 1e-3) / 1e12, "unit": UNIT,
                              "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
                              "ms_per_step": ms_per_step, "step_only": True, "launches_per_step": launches_per_step,
                              "config": {"workload": WORKLOAD_TEXT[headline]}}))
        return
    # the dominant kernel family (the bit-plane convolution) alone, in the step's output mode, cold L2, timed with
    # CUDA events on the launching stream while the clock sampler still runs
    mode = "fused" if chained else "raw"
    conv_graph = capture(lambda: [[L.run_conv(ebs, raw=not chained) for L in layers] for _ in range(inner)])
    conv_ms = timer.graph_ms(conv_graph, max(3, min(args.steps, 20)), cold=True) / inner
    clocks = sampler.stop()
    res["ms_per_step"] = ms_per_step
    res["binary_tops"] = total_ops / (ms_per_step * 1e-3) / 1e12
    res["int8_tops"] = total_int8 / (ms_per_step * 1e-3) / 1e12
    res["imgs_per_s"] = layers[0].n / (ms_per_step * 1e-3)

    # ---- end to end: pinned host codes in, the stack on the device, the last layer's packed planes back on the host
    first, last = layers[0], layers[-1]
    e2e = None
    if first.x is not None:
        x_host = first.x_host if first.x_host.is_pinned() else first.x_host.pin_memory()
        out_host = torch.empty(last.pn_bytes // 4, dtype=torch.int32).pin_memory()
        if chained:
            # Three streams, two buffers each for the network input, the last layer's planes and the host result:
            # the copy-in of step i+1 and the copy-out of step i-1 run under the kernels of step i.  Every step still
            # moves its own input in and its own result out; events order each buffer's reuse, and the host waits
            # for the result of step i-2 before that result's buffer is handed out again.
            torch.cuda.synchronize()
            pn_serial = last.pn.cpu()                           # the timed steps above ran the same input serially
            s_in, s_comp, s_out = (torch.cuda.Stream() for _ in range(3))
            xs, pns = [first.x, torch.empty_like(first.x)], [last.pn, torch.empty_like(last.pn)]
            outs = [out_host, torch.empty_like(out_host).pin_memory()]
            ev_in, ev_packed, ev_comp, ev_out = ([torch.cuda.Event() for _ in range(2)] for _ in range(4))
            counter = [0]

            def bound(b, fn):
                first.x, last.pn = xs[b], pns[b]
                return capture(fn)
            # the launches of one step as two graphs per buffer pair (the pack, then the 52 convolutions)
            pack_graphs = [bound(b, lambda: first.run_pack(ebs)) for b in range(2)]
            conv_graphs = [bound(b, lambda: [L.run_conv(ebs, raw=False) for L in layers]) for b in range(2)]

            def e2e_step():
                b = counter[0] & 1
                counter[0] += 1
                ev_out[b].synchronize()                         # the host has the result that last used outs[b]
                with torch.cuda.stream(s_in):
                    s_in.wait_event(ev_packed[b])               # ebs_pack_acts of two steps ago has read xs[b]
                    xs[b].copy_(x_host, non_blocking=True)
                    ev_in[b].record(s_in)
                with torch.cuda.stream(s_comp):
                    s_comp.wait_event(ev_in[b])
                    pack_graphs[b].replay()
                    ev_packed[b].record(s_comp)
                    conv_graphs[b].replay()                     # pns[b] is free: ev_out[b] was waited for on the host
                    ev_comp[b].record(s_comp)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_comp[b])
                    outs[b].copy_(pns[b], non_blocking=True)
                    ev_out[b].record(s_out)

            def e2e_drain():
                for s_ in (s_in, s_comp, s_out):
                    s_.synchronize()
                first.x, last.pn = xs[0], pns[0]
                # both buffers carry the result of the same input: the overlap lost or tore nothing
                if not (torch.equal(outs[0], outs[1]) and torch.equal(outs[0], pns[0].cpu())
                        and torch.equal(outs[0], pn_serial)):
                    raise RuntimeError("end-to-end leg: the overlapped steps disagree with the serial step")
            h2d, d2h = x_host.numel(), last.pn_bytes
            note = ("pinned u8 NHWC codes of the network input copied in, ebs_pack_acts, the 52 chained ebs_conv2d_mixed "
                    "calls (replayed as CUDA graphs), the last layer's packed planes copied back to pinned memory, every step; copies of "
                    "neighbouring steps overlap the kernels (3 streams, 2 buffers each); wall clock over the steps, "
                    "drained at the end")
        else:
            hosts = [(L, (L.x_host if L.x_host.is_pinned() else L.x_host.pin_memory()),
                      torch.empty(L.pn_bytes // 4, dtype=torch.int32).pin_memory()) for L in layers]
            ws = [torch.empty(max(ebs.ebs_host_workspace_bytes(L.d, L.n, L.spec.layer.h_in, L.spec.layer.w_in,
                                                               ebs.EBS_U8_CODES, L.next_bits) for L in layers),
                              dtype=torch.uint8, device=dev) for _ in range(3)]
            streams = [torch.cuda.Stream() for _ in range(3)]

            def e2e_step():
                for i, (L, xh, ph) in enumerate(hosts):
                    lay = L.spec.layer
                    ebs.ebs_conv2d_mixed_host(xh, ebs.EBS_U8_CODES, ebs.EBS_NHWC, L.n, lay.h_in, lay.w_in, L.pw, L.d,
                                              L.epi, ws[i % 3], None, None, ph, stream=streams[i % 3])
                for s_ in streams:
                    s_.synchronize()

            def e2e_drain():
                pass
            h2d, d2h = sum(xh.numel() for _, xh, _ in hosts), sum(L.pn_bytes for L in layers)
            note = ("ebs_conv2d_mixed_host per layer (independent inputs): pinned u8 codes in, packed next-layer planes "
                    "out; layers round-robin on 3 streams; wall clock")
        e2e_steps = max(3, min(args.steps, 20))
        for _ in range(3):
            e2e_step()
        e2e_drain()
        torch.cuda.synchronize()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        e2e_drain()
        e2e_s = max_over_ranks(time.perf_counter() - t0, dev) / e2e_steps
        e2e = {"value": world * total_ops / e2e_s / 1e12, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_s * 1e3, "note": note}

    if rank != 0:
        return
    peak_tops, hbm_gbs = int8_tensor_peak_tops(peaks), float(peaks.get("hbm_gbs", 6650.0))
    sm_max = float(clocks.get("sm_max_mhz") or sm_max)
    probes = {}
    if world == 1:
        try:
            probes = {"imma_mma_sync_tops": 2 * ebs.ebs_probe_pipe(3, 500) / 1e12,
                      "b1_mma_sync_tops": 2 * ebs.ebs_probe_pipe(1, 200) / 1e12,
                      "and_popc_add_tops": 2 * ebs.ebs_probe_pipe(0, 500) / 1e12,
                      # the instruction the conv kernels issue, from shared memory, nothing else running on the SM
                      "tcgen05_i8_m128n256k32_tops": 2 * ebs.ebs_probe_pipe(4, 2000) / 1e12}
        except Exception as exc:                                 # the probes are context, never fatal
            probes = {"error": str(exc)}
    # Roofline of the headline: the tensor-pipe kernels merge the planes of a channel back into one byte, so one
    # int8 multiply-accumulate retires all Wb*Ab plane pairs of that channel: the work the pipe executes is
    # 2*MACs int8 ops per layer, held against the int8 peak; a layer's roof is the slower of that and its packed
    # operand + output bytes at HBM bandwidth.  `bound` is whichever sum over the layers is larger.
    m = res["modes"][mode]
    if m["bound"] == "tensor":
        achieved, roof_peak, roof_unit = total_int8 / (conv_ms * 1e-3) / 1e12, peak_tops, "TOPS"
    else:
        achieved, roof_peak, roof_unit = m["algorithmic_bytes"] / (conv_ms * 1e-3) / 1e9, hbm_gbs, "GB/s"
    streaming = streaming_leg(ebs, dev, stream, hbm_gbs) if world == 1 and not args.quick else {}
    network = network_leg(ebs, dev, stream, flush, max(5, min(args.steps, 30))) if world == 1 and not args.quick else {}
    if network:
        network["resnet18_imagenet"] = resnet18_leg(ebs, dev, stream, flush, max(3, min(args.steps, 10)))
    cpu = cpu_baseline_sample(headline, 15.0) if world == 1 and not args.no_cpu_baseline else None
    res_head = dict(res)
    per_config[headline] = res_head
    line = {
        "metric": METRIC, "value": world * total_ops / (ms_per_step * 1e-3) / 1e12, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[headline], "global_batch": layers[0].n * world,
                   "imgs_per_s": world * layers[0].n / (ms_per_step * 1e-3),
                   "l2": "256 MB buffer rewritten before every timed step (cold L2)",
                   "launch": "each step is one CUDA-graph replay of its %d kernel launches" % launches_per_step,
                   "step": res["step"], "requantization": "per-layer steps calibrated once before timing (99.5th "
                                                          "percentile of the ReLU output onto the top code)" if chained
                   else "step 4*s_w*s_a*c_in per layer",
                   "parallelism": f"dp{world} (batch replicas, no data-path collective)"},
        "clocks": clocks,
        "gpu_launches": launches_per_step * args.steps * inner, "device_wait_timeouts": ebs.ebs_device_wait_timeouts(),
        "roofline": {"bound": m["bound"],
                     "kernel": "bit-plane conv, the %d launches of a step (tcgen05 kernels; planes merged to bytes on "
                               "chip), output mode of the step: %s" % (len(layers), m["outputs"]),
                     "achieved": achieved, "peak": roof_peak, "unit": roof_unit, "frac": achieved / roof_peak,
                     "traffic": ncu_traffic_per_launch(headline),
                     "accounting": "achieved = executed int8 ops (2*MACs: one byte multiply-accumulate retires all "
                                   "Wb*Ab plane pairs of a channel) of the conv launches / their CUDA-event time when the "
                                   "layers' tensor roofs sum to more than their HBM roofs, else algorithmic bytes (packed "
                                   "input planes + weight byte image + requested outputs) / time",
                     "conv_ms_per_step": conv_ms, "conv_launches_per_step": len(layers),
                     "avg_launch_us": conv_ms * 1e3 / len(layers),
                     "effective_binary_tops_conv": total_ops / (conv_ms * 1e-3) / 1e12,
                     "int8_tops_conv": total_int8 / (conv_ms * 1e-3) / 1e12,
                     "gbs_conv": m["algorithmic_bytes"] / (conv_ms * 1e-3) / 1e9,
                     "tensor_peak_tops": peak_tops, "hbm_peak_gbs": hbm_gbs,
                     # context: the same work against the rate the library's own tcgen05 int8 probe reaches on this GPU
                     "frac_of_tcgen05_i8_probe": (total_int8 / (conv_ms * 1e-3) / 1e12 / probes["tcgen05_i8_m128n256k32_tops"]
                                                  if probes.get("tcgen05_i8_m128n256k32_tops") else None),
                     "peak_source": f"hbm_gbs {hbm_gbs} ({peak_kind}); int8 dense = 2 x bf16 burst "
                                    f"({peaks.get('bf16_tflops')} TFLOP/s, {peak_kind})",
                     "sum_layer_roofs_ms": m["sum_layer_roofs_ms"],
                     "frac_of_layer_roofs_cold": m["sum_layer_roofs_ms"] / conv_ms,
                     "frac_of_layer_roofs_warm": m["frac_of_layer_roofs"],
                     "other_pipes": dict(probes, popc_pipe_unit_count_tops=popc_pipe_peak_tops(sm_max)),
                     "per_layer_note": "per-layer times are L2-warm (10 back-to-back launches in a graph); roof = "
                                       "max(2*MACs / int8 tensor peak, algorithmic bytes / HBM peak); see per_config"},
        "literal_bitplane_path": dict(res["literal_bitplane_path"],
                                      note="every bit pair is one AND+POPC lane-op here, so binary ops are what this "
                                           "pipe executes; the default path retires Wb*Ab of them per int8 MAC"),
        "per_config": per_config,
        "streaming_kernels": streaming,
        "network": network,
        "wall_s_timed_region": wall,
    }
    if e2e is not None:
        line["e2e"] = e2e
    if cpu is not None:
        line["cpu_baseline"] = cpu
        per_config[headline]["cpu_baseline"] = cpu
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true", help="skip the streaming-kernel and whole-network legs")
    ap.add_argument("--step-only", action="store_true",
                    help="time the steps of --workload and print a short line: no per-layer, per-mode or context legs "
                         "(the command profiler captures run)")
    ap.add_argument("--workload", default="all", choices=["all"] + sorted(WORKLOAD_TEXT),
                    help="all (default): the five configurations, headline config5; configN: that one alone")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
