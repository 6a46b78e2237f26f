#!/usr/bin/env python
"""Benchmark of the bit-plane mixed-precision convolution path on the CIFAR ResNet-20 stack.

A step is one pass of the whole path over one batch of 128 synthetic images: for each of the 20
quantized convolution layers, activation quantize+pack (ebs_pack_acts), the bit-plane convolution
with fused epilogue writing int32 accumulators and the next layer's packed planes
(ebs_conv2d_mixed), and the stand-alone de-quantization (ebs_dequant).  Weight packing is done once
before timing (it is off the inference path).  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
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

import numpy as np  # noqa: E402
import torch  # noqa: E402

from workloads import gen  # noqa: E402

METRIC = "effective binary TOPS (2*MACs*Wb*Ab per second), ResNet-20 CIFAR quantized conv stack"
UNIT = "TOPS"
WORKLOAD = "config2: ResNet-20 CIFAR-shaped stack, 20 quantized convs, batch 128, (Wb,Ab) in {1..4}^2, seed 0"
# other workloads of the same path, for profiling and for the results table (the default is config2)
WORKLOADS = {
    "config2": (WORKLOAD, lambda: [s for s in gen.config2(0) if s.layer.quantized]),
    "config1": ("config1: one 3x3 conv 64->64, 32x32, batch 1, W2A2, seed 0", lambda: gen.config1(0)),
    "config3": ("config3: ResNet-18 ImageNet-shaped quantized convs, batch 64, (Wb,Ab) in {2..6}^2, seed 0",
                lambda: gen.config3(0)),
    "config4": ("config4: 4096^3 bit-plane GEMM as a 1x1 convolution over 64x64 pixels, seven (Wb,Ab) pairs of the sweep, seed 0",
                lambda: [gen.config4(wb, ab) for wb, ab in [(1, 1), (2, 2), (4, 4), (8, 8), (1, 8), (8, 1), (3, 5)]]),
    "config5": ("config5: ResNet-50 ImageNet-shaped bottleneck stack, batch 256, (Wb,Ab) in {2..8}^2, seed 0 "
                "(layers run with independent inputs here; the chained run is a parity test)",
                lambda: gen.config5(0)),
}
SM_COUNT, POPC_LANES_PER_CLK_SM = 148, 16
# dram__bytes_read.sum + dram__bytes_write.sum per conv launch, mean over the 20 layers, from the ncu
# capture summarised in profiles/ (outputs stay in the 126 MB L2 while ncu replays a launch)
NCU_TRAFFIC_BYTES_PER_LAUNCH = 689207


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "sm_max_mhz": 1965.0}, "fallback"


def int8_tensor_peak_tops(peaks: dict) -> float:
    """Dense int8 tensor peak in TOPS: the measured bf16 burst figure times the nominal int8:bf16 ratio (2)."""
    return 2.0 * float(peaks.get("bf16_tflops", 1590.0))


def hbm_gbs_for_streaming(peaks: dict) -> float:
    return float(peaks.get("hbm_gbs", 6650.0))


def popc_pipe_peak_tops(sm_max_mhz: float) -> float:
    """Binary TOPS of the POPC pipe: 16 lanes/clk/SM x 32 bit x 148 SMs x clock, 2 ops per bit pair."""
    return 2.0 * SM_COUNT * POPC_LANES_PER_CLK_SM * 32 * sm_max_mhz * 1e6 / 1e12


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


# ---------------------------------------------------------------------------- GPU arm

class Layer:
    """Device buffers and descriptors of one layer (plumbing only)."""

    def __init__(self, ebs, spec, next_bits, dev):
        L = spec.layer
        self.spec, self.n, self.next_bits = spec, spec.batch, next_bits
        self.d = ebs.conv_desc(L.c_in, L.c_out, L.k, L.k, L.stride, L.stride, L.pad, L.pad, spec.w_bits, spec.a_bits,
                               spec.w_scale, spec.a_scale)
        qa = gen.act_codes(spec).astype(np.uint8)
        self.x_host = torch.from_numpy(np.ascontiguousarray(qa.transpose(0, 2, 3, 1))).pin_memory()   # NHWC codes
        self.x = self.x_host.to(dev)
        qw = torch.from_numpy(gen.weight_codes(spec).astype(np.int8)).to(dev)
        self.pw = torch.empty(ebs.ebs_packed_weight_bytes(self.d) // 4, dtype=torch.int32, device=dev)
        ebs.ebs_pack_weights(qw, ebs.EBS_I8_CODES, ebs.EBS_NCHW, self.d, self.pw)
        self.px = torch.empty(ebs.ebs_packed_act_bytes(self.n, L.h_in, L.w_in, L.c_in, spec.a_bits) // 4,
                              dtype=torch.int32, device=dev)
        ho, wo = L.h_out, L.w_out
        self.pixels = self.n * ho * wo
        self.acc = torch.empty((self.n, ho, wo, L.c_out), dtype=torch.int32, device=dev)
        self.y = torch.empty((self.n, ho, wo, L.c_out), dtype=torch.float32, device=dev)
        self.pn_bytes = ebs.ebs_packed_act_bytes(self.n, ho, wo, L.c_out, next_bits)
        self.pn = torch.empty(self.pn_bytes // 4, dtype=torch.int32, device=dev)
        self.pn_host = torch.empty(self.pn_bytes // 4, dtype=torch.int32).pin_memory()
        self.epi = ebs.epilogue(relu=True, next_a_bits=next_bits, next_a_scale=4.0 * spec.w_scale * spec.a_scale * L.c_in)
        self.S = float(np.float32(spec.w_scale) * np.float32(spec.a_scale))
        self.ops = gen.binary_ops(spec)
        self.ws_bytes = ebs.ebs_host_workspace_bytes(self.d, self.n, L.h_in, L.w_in, ebs.EBS_U8_CODES, next_bits)

    def run_pack(self, ebs):
        L = self.spec.layer
        ebs.ebs_pack_acts(self.x, ebs.EBS_U8_CODES, ebs.EBS_NHWC, self.n, L.c_in, L.h_in, L.w_in, self.spec.a_bits,
                          self.spec.a_scale, self.px)

    def run_dequant(self, ebs):
        ebs.ebs_dequant(self.acc, self.pixels, self.spec.layer.c_out, self.S, None, None, True, self.y)

    def run_conv_only(self, ebs, variant=-1):
        L = self.spec.layer
        ebs.ebs_conv2d_mixed(self.px, self.n, L.h_in, L.w_in, self.pw, self.d, self.epi, self.acc, None, self.pn,
                             variant=variant)

    def run_host(self, ebs, ws, stream=None):
        L = self.spec.layer
        ebs.ebs_conv2d_mixed_host(self.x_host, ebs.EBS_U8_CODES, ebs.EBS_NHWC, self.n, L.h_in, L.w_in, self.pw, self.d,
                                  self.epi, ws, None, None, self.pn_host, stream=stream)


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


class OracleWorkload:
    """The CPU oracle on (a batch slice of) the same workload; codes are generated outside the timing."""

    def __init__(self, batch: int):
        import oracle
        oracle.build()
        self.oracle, self.batch = oracle, batch
        self.specs = [s for s in gen.config2(0) if s.layer.quantized]
        self.data = [(gen.act_codes(s, batch=batch), gen.weight_codes(s)) for s in self.specs]
        self.ops = sum(gen.binary_ops(s, batch=batch) for s in self.specs)

    def step(self) -> float:
        t0 = time.perf_counter()
        for s, (qa, qw) in zip(self.specs, self.data):
            L = s.layer
            acc = self.oracle.conv2d_codes(qa, qw, (L.stride, L.stride), (L.pad, L.pad))
            self.oracle.epilogue(acc, self.oracle.combined_scale(s.w_scale, s.a_scale), relu=True)
        return time.perf_counter() - t0


def oracle_batch_for(budget_s: float, n_steps: int) -> int:
    """Largest batch (<= 128) for which n_steps oracle passes fit the time budget."""
    probe = OracleWorkload(2)
    probe.step()
    per_image = probe.step() / 2
    return int(max(1, min(128, budget_s / max(n_steps, 1) / per_image)))


def cpu_baseline_sample(budget_s: float = 15.0):
    """The oracle, as it stands, timed on this host's cores on a bounded sample (a reported baseline)."""
    wl = OracleWorkload(oracle_batch_for(budget_s, 3))
    wl.step()
    times = [wl.step() for _ in range(2)]
    dt = float(np.mean(times))
    return {"value": wl.ops / dt / 1e12, "unit": UNIT, "cores": wl.oracle.num_threads(), "kind": "oracle",
            "sample": f"all 20 quantized layers at batch {wl.batch} of 128 (direct integer conv + fp32 epilogue), "
                      f"mean of 2 passes of {dt:.2f} s"}


def run_reference(args):
    rank, world, _ = dist_setup(args.gpus)
    if rank != 0:
        return
    wl = OracleWorkload(oracle_batch_for(150.0, args.steps + args.warmup))
    for _ in range(args.warmup):
        wl.step()
    times = [wl.step() for _ in range(args.steps)]
    dt = float(np.mean(times))
    value = wl.ops / dt / 1e12
    base = {"value": value, "unit": UNIT, "cores": wl.oracle.num_threads(), "kind": "oracle",
            "sample": f"each step: all 20 quantized layers at batch {wl.batch} of 128"}
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample_batch": wl.batch},
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def network_leg(ebs, dev, stream, flush, capture, reps):
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


def run_gpu(args):
    from paper_2003_07577_b200 import binding as ebs
    ebs.lib()
    rank, world, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    peaks, peak_kind = measured_peaks()

    workload_text, make_specs = WORKLOADS[args.workload]
    specs = make_specs()                                            # every rank: one full batch (weak scaling)
    if args.only:                                                   # profiling aid: a subset of the layers
        specs = [s for s in specs if s.layer.name in args.only.split(",")]
    layers = [Layer(ebs, s, specs[(i + 1) % len(specs)].a_bits, dev) for i, s in enumerate(specs)]
    ws = torch.empty(max(L.ws_bytes for L in layers), dtype=torch.uint8, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > 126 MB L2
    total_ops = sum(L.ops for L in layers)
    stream = torch.cuda.current_stream()

    def one_step():
        # the path as a network runs it: activations are quantized and packed once, at the entry (row a2); every
        # layer is one fused launch whose epilogue writes the int32 accumulators and the next layer's planes
        # (rows a3-a5); the accumulators are de-quantized once, at the exit (row a6)
        layers[0].run_pack(ebs)
        for L in layers:
            L.run_conv_only(ebs)
        layers[-1].run_dequant(ebs)

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

    for L in layers:                                                # every layer's resident planes (set-up, untimed)
        L.run_pack(ebs)
    for _ in range(max(args.warmup, 3)):
        one_step()
    torch.cuda.synchronize()
    step_graph = capture(one_step)
    conv_graph = capture(lambda: [L.run_conv_only(ebs) for L in layers])
    for _ in range(3):
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
    step_ms = [e0.elapsed_time(e1) for e0, e1 in ev]
    total_ms = max_over_ranks(float(sum(step_ms)), dev)
    ms_per_step = total_ms / args.steps

    # dominant kernel (the bit-plane convolution) alone: the 20 conv launches of a step, cold L2 per replay
    reps = max(3, min(args.steps, 20))
    cev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for e0, e1 in cev:
        flush.zero_()
        e0.record(stream)
        conv_graph.replay()
        e1.record(stream)
    torch.cuda.synchronize()
    conv_total_ms = float(np.mean([e0.elapsed_time(e1) for e0, e1 in cev]))
    clocks = sampler.stop()

    # per-layer breakdown: each layer's conv launched 10 times back to back in a graph (L2-warm)
    conv_ms = np.zeros(len(layers))
    for i, L in enumerate(layers):
        g = capture(lambda L=L: [L.run_conv_only(ebs) for _ in range(10)])
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g.replay()
        e0.record(stream)
        g.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        conv_ms[i] = e0.elapsed_time(e1) / 10.0

    # the same 20 conv launches on the integer-pipe kernels only: the plane-pair double sum evaluated
    # literally (AND + POPC + shift-add per plane pair), held against the POPC pipe's peak
    literal = {}
    if world == 1:
        lit_graph = capture(lambda: [L.run_conv_only(ebs, -2) for L in layers])
        lev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for e0, e1 in lev:
            flush.zero_()
            e0.record(stream)
            lit_graph.replay()
            e1.record(stream)
        torch.cuda.synchronize()
        lit_ms = float(np.mean([e0.elapsed_time(e1) for e0, e1 in lev]))
        literal = {"kernel": "conv_popc_kernel (variant -2: the library's choice among the integer-pipe kernels)",
                   "conv_ms_per_step": lit_ms, "binary_tops": total_ops / (lit_ms * 1e-3) / 1e12}

    # the streaming kernels (rows a2 and a6) on a tensor far larger than L2: achieved GB/s of algorithmic bytes
    streaming = {}
    if world == 1:
        sn, sh, sc, sab = 256, 56, 64, 4                                   # ResNet-50 layer-1 activations: 51 M values, inputs > L2
        vals = sn * sh * sh * sc
        xf = torch.rand((sn, sh, sh, sc), dtype=torch.float32, device=dev)
        xu = torch.randint(0, 16, (sn, sh, sh, sc), dtype=torch.uint8, device=dev)
        pk = torch.empty(ebs.ebs_packed_act_bytes(sn, sh, sh, sc, sab) // 4, dtype=torch.int32, device=dev)
        ai = torch.randint(-1000, 1000, (sn * sh * sh, sc), dtype=torch.int32, device=dev)
        yo = torch.empty((sn * sh * sh, sc), dtype=torch.float32, device=dev)

        def gbs(fn, nbytes, reps=10):
            fn()
            tot = 0.0
            for _ in range(reps):                                       # inputs are larger than L2: no flush needed
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                torch.cuda.synchronize()
                tot += a.elapsed_time(b)
            return nbytes / (tot / reps * 1e-3) / 1e9

        out_b = vals * sab // 8
        streaming = {
            "tensor": f"{sn}x{sh}x{sh}x{sc} NHWC, {sab} planes", "hbm_peak_gbs": hbm_gbs_for_streaming(peaks),
            "pack_acts_fp32_gbs": gbs(lambda: ebs.ebs_pack_acts(xf, ebs.EBS_F32, ebs.EBS_NHWC, sn, sc, sh, sh, sab, 0.07, pk),
                                      vals * 4 + out_b),
            "pack_acts_u8_gbs": gbs(lambda: ebs.ebs_pack_acts(xu, ebs.EBS_U8_CODES, ebs.EBS_NHWC, sn, sc, sh, sh, sab, 1.0, pk),
                                    vals + out_b),
            "pack_acts_fp32_nchw_gbs": gbs(lambda: ebs.ebs_pack_acts(xf, ebs.EBS_F32, ebs.EBS_NCHW, sn, sc, sh, sh, sab, 0.07, pk),
                                           vals * 4 + out_b),
            "dequant_gbs": gbs(lambda: ebs.ebs_dequant(ai, sn * sh * sh, sc, 0.01, None, None, True, yo), vals * 8),
        }
        # search-stage forward (Eq. 6-7), five candidate bitwidths: 4 B in + 4 B out per value; the weight form
        # reads the tensor once more for max|w|
        cand_bits, cand_coeff = [1, 2, 3, 4, 5], [0.1, 0.15, 0.4, 0.25, 0.1]
        scratch = torch.zeros(4, dtype=torch.int32, device=dev)
        xo = torch.empty_like(xf)
        streaming["search_act_forward_gbs"] = gbs(lambda: ebs.ebs_search_act_forward(xf, 6.0, cand_bits, cand_coeff, xo), vals * 8)
        streaming["search_weight_forward_gbs"] = gbs(
            lambda: ebs.ebs_search_weight_forward(xf, cand_bits, cand_coeff, xo, scratch), vals * 12)
        del xo
        del xf, xu, pk, ai, yo

    # whole-network inference (the ResNet-20 of this workload wired with its shortcuts, pooling and
    # classifier): one CUDA-graph replay per batch, cold L2; and the same from pinned host images to
    # host logits
    network = {}
    if world == 1 and args.workload == "config2" and not args.only:
        network = network_leg(ebs, dev, stream, flush, capture, max(5, min(args.steps, 30)))

    # end to end through the host entry point: pinned host codes in, packed planes out, every step
    # The layers of this workload have independent inputs, so they are issued round-robin on three
    # streams (each with its own workspace): the upload of one layer overlaps the kernels of another
    # and the download of a third.
    e2e_steps = max(3, min(args.steps, 10))
    e2e_streams = [torch.cuda.Stream() for _ in range(3)]
    e2e_ws = [ws] + [torch.empty_like(ws) for _ in range(len(e2e_streams) - 1)]

    def e2e_step():
        for i, L in enumerate(layers):
            k = i % len(e2e_streams)
            L.run_host(ebs, e2e_ws[k], e2e_streams[k])
        for st_ in e2e_streams:
            st_.synchronize()

    e2e_step()
    torch.cuda.synchronize()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    e2e_s = max_over_ranks(time.perf_counter() - t0, dev) / e2e_steps

    if rank != 0:
        return
    sm_max = float(clocks.get("sm_max_mhz") or peaks.get("sm_max_mhz", 1965.0))
    peak_tops = int8_tensor_peak_tops(peaks)                 # 1 bit-pair AND+bitcount = 1 byte MAC = 2 ops
    hbm_gbs = float(peaks.get("hbm_gbs", 6650.0))
    probes = {}
    if world == 1:
        try:
            probes = {"imma_mma_sync_tops": 2 * ebs.ebs_probe_pipe(3, 500) / 1e12,
                      "b1_mma_sync_tops": 2 * ebs.ebs_probe_pipe(1, 200) / 1e12,
                      "and_popc_add_tops": 2 * ebs.ebs_probe_pipe(0, 500) / 1e12}
        except Exception as exc:                                 # the probes are context, never fatal
            probes = {"error": str(exc)}
    # Roofline accounting.  The tensor-pipe kernels merge the planes of a channel back into one byte, so one
    # int8 multiply-accumulate retires all Wb*Ab plane pairs of that channel: the work the pipe executes is
    # 2*MACs int8 ops per layer (not 2*MACs*Wb*Ab), and that is what is held against the int8 peak.  A
    # layer's roof is the slower of that and its packed operand + output bytes at HBM bandwidth.
    per_layer, roof_ms, sum_tensor_s, sum_hbm_s, sum_bytes, sum_int8_ops = [], 0.0, 0.0, 0.0, 0, 0
    for L, t in zip(layers, conv_ms):
        lay = L.spec.layer
        bytes_alg = (L.px.numel() * 4 + ebs.ebs_packed_weight_plane_bytes(L.d) + L.acc.numel() * 4 + L.pn_bytes)
        int8_ops = L.ops // (L.spec.w_bits * L.spec.a_bits)                 # 2 * MACs
        t_tensor, t_hbm = int8_ops / (peak_tops * 1e12), bytes_alg / (hbm_gbs * 1e9)
        roof = max(t_tensor, t_hbm)
        roof_ms += roof * 1e3
        sum_tensor_s += t_tensor; sum_hbm_s += t_hbm; sum_bytes += bytes_alg; sum_int8_ops += int8_ops
        per_layer.append({"name": lay.name, "wb": L.spec.w_bits, "ab": L.spec.a_bits, "us": round(float(t) * 1e3, 2),
                          "tops": round(L.ops / (t * 1e-3) / 1e12, 1), "bytes": int(bytes_alg),
                          "int8_tops": round(int8_ops / (t * 1e-3) / 1e12, 1),
                          "roof_us": round(roof * 1e6, 2), "roof": "tensor" if t_tensor >= t_hbm else "hbm",
                          "frac_of_roof": round(roof * 1e3 / float(t), 3)})
    bound = "tensor" if sum_tensor_s >= sum_hbm_s else "hbm"
    if bound == "tensor":
        achieved, roof_peak, roof_unit = sum_int8_ops / (conv_total_ms * 1e-3) / 1e12, peak_tops, "TOPS"
    else:
        achieved, roof_peak, roof_unit = sum_bytes / (conv_total_ms * 1e-3) / 1e9, hbm_gbs, "GB/s"
    cpu = cpu_baseline_sample() if world == 1 and not args.no_cpu_baseline else None
    line = {
        "metric": METRIC, "value": world * total_ops / (ms_per_step * 1e-3) / 1e12, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": workload_text + (f" [only {args.only}]" if args.only else ""), "global_batch": specs[0].batch * world,
                   "imgs_per_s": world * specs[0].batch / (ms_per_step * 1e-3),
                   "l2": "256 MB buffer rewritten before every timed step (cold L2)",
                   "launch": "each step is one CUDA-graph replay of its %d kernel launches" % (len(layers) + 2),
                   "step": "ebs_pack_acts(u8 NHWC) at the entry, ebs_conv2d_mixed(acc + packed_next) per layer, "
                           "ebs_dequant at the exit; every layer reads its own resident synthetic planes",
                   "parallelism": f"dp{world} (batch replicas, no data-path collective)"},
        "clocks": clocks,
        "e2e": {"value": world * total_ops / e2e_s / 1e12, "unit": UNIT,
                "h2d_bytes_per_step": int(sum(L.x_host.numel() for L in layers)),
                "d2h_bytes_per_step": int(sum(L.pn_bytes for L in layers)),
                "note": "ebs_conv2d_mixed_host per layer: pinned u8 codes in, packed next-layer planes out; layers round-robin on 3 streams; wall clock"},
        "gpu_launches": (len(layers) + 2) * args.steps, "device_wait_timeouts": ebs.ebs_device_wait_timeouts(),
        "roofline": {"bound": bound,
                     "kernel": "bit-plane conv, the %d launches of a step (conv_umma_strip_kernel / conv_umma_resident_kernel "
                               "/ conv_umma_kernel: tcgen05; conv_mma_kernel / conv_mma_strip_kernel: mma.sync; planes "
                               "merged to bytes on chip)" % len(layers),
                     "achieved": achieved, "peak": roof_peak, "unit": roof_unit, "frac": achieved / roof_peak,
                     "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH if args.workload == "config2" and not args.only else None,
                     "accounting": "achieved = algorithmic bytes (packed input planes + weight planes + int32 accumulators "
                                   "+ packed output planes) of the conv launches / their time when the layers' HBM roofs "
                                   "sum to more than their tensor roofs, else executed int8 ops (2*MACs: one byte "
                                   "multiply-accumulate retires all Wb*Ab plane pairs of a channel) / time",
                     "effective_binary_tops_conv": total_ops / (conv_total_ms * 1e-3) / 1e12,
                     "int8_tops_conv": sum_int8_ops / (conv_total_ms * 1e-3) / 1e12,
                     "tensor_peak_tops": peak_tops,
                     "peak_source": f"hbm_gbs {hbm_gbs} ({peak_kind}); int8 dense = 2 x bf16 burst "
                                    f"({peaks.get('bf16_tflops')} TFLOP/s, {peak_kind})",
                     "conv_ms_per_step": conv_total_ms, "conv_launches_per_step": len(layers),
                     "algorithmic_bytes_per_launch": int(np.mean([pl["bytes"] for pl in per_layer])),
                     "sum_layer_roofs_ms": roof_ms, "frac_of_layer_roofs": roof_ms / float(conv_ms.sum()),
                     "hbm_peak_gbs": hbm_gbs, "hbm_peak_kind": peak_kind,
                     "other_pipes": dict(probes, popc_pipe_unit_count_tops=popc_pipe_peak_tops(sm_max)),
                     "per_layer_note": "per-layer times are L2-warm (10 back-to-back launches in a graph); "
                                       "roof = max(2*MACs / int8 tensor peak, algorithmic bytes / HBM peak)",
                     "per_layer": per_layer},
        "literal_bitplane_path": dict(literal, popc_pipe_peak_tops=popc_pipe_peak_tops(sm_max),
                                      frac_of_popc_pipe=(literal["binary_tops"] / popc_pipe_peak_tops(sm_max)
                                                         if literal else None),
                                      note="every bit pair is one AND+POPC lane-op here, so binary ops are what this "
                                           "pipe executes; the default path above retires Wb*Ab of them per int8 MAC"),
        "streaming_kernels": streaming,
        "network": network,
        "wall_s_timed_region": wall,
    }
    if cpu is not None:
        line["cpu_baseline"] = cpu
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="config2", choices=sorted(WORKLOADS), help="default: the bench workload")
    ap.add_argument("--only", default="", help="comma-separated layer names: restrict the step to these layers (for profiling)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
