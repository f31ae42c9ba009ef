#!/usr/bin/env python
"""Benchmark of the sub-bit binary 3x3 convolution library on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

One "step" is one pass of the whole hot path over one batch: the 16 binary 3x3
layers of the ImageNet ResNet-18-shaped stack (batch 64 per GPU, tau = 5,
bit-packed +/-1 activations), each layer on its own seeded synthetic input,
launched back to back on one stream through the C ABI.  Prints ONE JSON line.

With N > 1 (torchrun) every rank runs its own batch of 64 on its own GPU: the
images are independent, there is no exchange step, so the scaling is weak and
no collective is on the data path (only the timing reduction uses one).

`--impl reference` times the CPU oracle (oracle/, the plain nested-loop
definition) on the host cores on a bounded sample of the same workload.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "ResNet-18 binary conv-stack img/s (dense-equivalent binary-conv TOPS in effective_tops)"
UNIT = "img/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML while the timed region runs."""

    def __init__(self, device_index: int, period_s: float = 0.005):
        self.idx, self.period = device_index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = device_index
            if visible:
                ids = [v for v in visible.split(",") if v.strip()]
                if device_index < len(ids) and ids[device_index].strip().isdigit():
                    phys = int(ids[device_index])
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join(timeout=2)
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------------
# reference arm: the CPU oracle on the host cores
# --------------------------------------------------------------------------
def time_oracle_stack(workload, n_images: int, max_layers=None):
    """Runs n_images through every layer of the stack with the oracle; returns seconds."""
    import oracle
    t_total = 0.0
    for i, shape in enumerate(workload.layers[:max_layers]):
        seed = wl.layer_seed(workload.config, i)
        p = wl.draw_layer_params(shape, workload.tau, seed)
        if workload.act == "bin" and shape.ksize == 1:
            act = wl.pack_activation_bits(wl.draw_activation_bits(shape, n_images, seed))
            t0 = time.perf_counter()
            oracle.conv1x1_bin(p.codebook, workload.tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride, act)
            t_total += time.perf_counter() - t0
        elif workload.act == "bin":
            act = wl.pack_activation_bits(wl.draw_activation_bits(shape, n_images, seed))
            t0 = time.perf_counter()
            oracle.conv_bin(p.codebook, workload.tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride,
                            shape.pad, act)
            t_total += time.perf_counter() - t0
        else:
            act = wl.draw_activation_f16(shape, n_images, seed)
            t0 = time.perf_counter()
            oracle.conv_f16(p.codebook, workload.tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out, shape.stride,
                            shape.pad, act)
            t_total += time.perf_counter() - t0
    return t_total


def oracle_sample_images(workload, budget_s: float = 15.0) -> int:
    """Images per step so that one oracle pass over the stack takes about budget_s."""
    import oracle
    oracle.build()
    t1 = time_oracle_stack(workload, 1)
    n = int(max(1, min(workload.batch, budget_s / max(t1, 1e-6))))
    return n


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    workload = wl.get_workload(args.workload)
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    # bound the whole run to a few minutes: at most ~120 s of oracle time in total
    per_step_budget = max(1.0, min(15.0, 120.0 / (steps + warmup)))
    n_img = oracle_sample_images(workload, per_step_budget)
    for _ in range(warmup):
        time_oracle_stack(workload, n_img)
    t = 0.0
    for _ in range(steps):
        t += time_oracle_stack(workload, n_img)
    ms = t / steps * 1e3
    value = n_img / (ms * 1e-3)
    cores = oracle.threads()
    sample = f"{n_img} of {workload.batch} images through all {len(workload.layers)} layers per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int32" if workload.act == "bin" else "f64", "data": "synthetic",
        "config": {"workload": _workload_name(workload), "images_per_step": n_img},
        "effective_tops": 2 * workload.with_batch(n_img).dense_macs() / (ms * 1e-3) / 1e12,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# DRAM traffic per launch of the dominant kernel from an ncu capture (profiles/), valid only while
# the kernel's sources are the ones that were profiled: {kernel: (workload, batch, bytes, sha256 of sources)}
_TRAFFIC = {
    # profiles/dram_traffic_resnet18_stack_n64_grouped.txt: mean of the two captured launches
    "tcg_conv_kernel (grouped decoded_tc)": ("resnet18", 64, 351645312,
                                             "80cb07752f0febac30141a098d3da70cbee8f49414eaad1867e0df037338bf63"),
}


def _kernel_fingerprint():
    """sha256 of the tensor-core kernel's sources with comments and blank space removed: it changes when the code does."""
    import hashlib
    import re
    h = hashlib.sha256()
    for f in ("snn_tcg.cu", "snn_tc_common.cuh"):
        with open(os.path.join(ROOT, "paper_2110_09195_b200", "csrc", f), "r") as fh:
            text = re.sub(r"//[^\n]*", "", fh.read())
        h.update("".join(text.split()).encode())
    return h.hexdigest()


def _profiled_traffic(kernel_name, nb, workload):
    rec = _TRAFFIC.get(kernel_name)
    if rec is None or rec[0] != workload.name or rec[1] != nb:
        return None
    return rec[2] if _kernel_fingerprint() == rec[3] else None


def _workload_name(workload):
    return f"{workload.name}_stack_n{workload.batch}_tau{workload.tau}_{workload.act}"


_SKEWS = {"none": None, "deep": wl.SKEW_DEEP, "top64": wl.SKEW_TOP64}


# --------------------------------------------------------------------------
# own arm
# --------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2110_09195_b200 as snn
    from paper_2110_09195_b200 import replicas

    info = replicas.rank_info()
    rank, world, local_rank = info.rank, info.world, info.local_rank
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    snn.load_library()
    peaks = _peaks()
    workload = wl.get_workload(args.workload, tau=args.tau, batch=args.batch)
    first_layer = 0
    if args.layers:
        lo, hi = (int(v) for v in args.layers.split(":"))
        first_layer = lo
        workload = wl.Workload(workload.name + f"[{lo}:{hi}]", workload.config, workload.batch, workload.tau,
                               workload.act, workload.layers[lo:hi])
    nb = workload.batch
    skew = _SKEWS[args.index_skew]
    act_code = snn.ACT_BIN if workload.act == "bin" else snn.ACT_F16
    forced = {"auto": snn.PATH_AUTO, "reuse": snn.PATH_REUSE, "decoded": snn.PATH_DECODED,
              "decoded_tc": snn.PATH_DECODED_TC}[args.path]

    layers, acts, outs, host_acts, host_outs, paths, params = [], [], [], [], [], [], []
    for i, shape in enumerate(workload.layers, start=first_layer):
        seed = wl.layer_seed(workload.config, i) + 7919 * rank
        p = wl.draw_layer_params(shape, workload.tau, wl.layer_seed(workload.config, i), index_skew=skew)
        layer = snn.SnnConv(shape.c_in, shape.c_out, workload.tau, p.codebook, p.idx_packed, p.alpha, shape.stride,
                            shape.pad, act_code, device=local_rank, ksize=shape.ksize)
        if workload.act == "bin":
            a = torch.from_numpy(wl.pack_activation_bits(wl.draw_activation_bits(shape, nb, seed)).view(np.int32))
        else:
            a = torch.from_numpy(wl.draw_activation_f16(shape, nb, seed))
        host_acts.append(a.pin_memory())
        acts.append(a.to(dev))
        outs.append(layer.alloc_out(nb, shape.h, shape.w))
        host_outs.append(layer.alloc_out(nb, shape.h, shape.w, pin=True))
        if forced == snn.PATH_AUTO and not args.group_only:
            layer.tune(nb, shape.h, shape.w)
        paths.append(layer.chosen_path(nb, shape.h, shape.w) if forced == snn.PATH_AUTO else forced)
        layers.append(layer)
        params.append(p)

    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)  # > 126 MB L2
    side = torch.cuda.Stream(dev)
    stream = torch.cuda.current_stream(dev)
    all_idx = list(range(len(layers)))
    use_graph = not args.no_graph

    def launch_layers(idxs, s):
        for j in idxs:
            layers[j].forward(acts[j], outs[j], snn.OUT_F32, paths[j], s)

    def as_graph(fn):
        """The launches of `fn(stream)` as a CUDA graph, so that the host's per-call cost does not sit between
        the kernels that are being timed."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            fn(side)                       # warm-up outside capture (sets kernel attributes, builds plans)
            side.synchronize()
            with torch.cuda.graph(g, stream=side):
                fn(torch.cuda.current_stream(dev))
        return g

    def timed(fn, steps, warm=3):
        """Median-free mean of `steps` device-timed runs of fn(), L2 flushed before each (outside the events)."""
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(steps + warm):
            flush.zero_()
            if i >= warm:
                ev[i - warm][0].record(stream)
            fn()
            if i >= warm:
                ev[i - warm][1].record(stream)
        torch.cuda.synchronize(dev)
        return float(sum(a.elapsed_time(b) for a, b in ev)) / steps

    group = None
    grouped = not args.per_layer and forced in (snn.PATH_AUTO, snn.PATH_DECODED_TC)
    if grouped:
        # The layers of the benchmark are independent problems (each has its own input): the step
        # is one persistent launch that walks through all of them (snn_conv_group_forward).
        group = snn.SnnConvGroup(layers, [(nb, s.h, s.w) for s in workload.layers])
        step_graph = as_graph(lambda s: group.forward(acts, outs, snn.OUT_F32, s)) if use_graph else None
        step_host = lambda: group.forward(acts, outs, snn.OUT_F32, stream)   # noqa: E731
    else:
        step_graph = as_graph(lambda s: launch_layers(all_idx, s)) if use_graph else None
        step_host = lambda: launch_layers(all_idx, stream)                    # noqa: E731

    def step():
        if use_graph:
            step_graph.replay()
        else:
            step_host()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(max(3, args.warmup)):
        flush.zero_()
        step()
    barrier()

    sampler = ClockSampler(local_rank)
    sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    launches0 = snn.kernel_launches()
    barrier()
    wall0 = time.perf_counter()
    for e0, e1 in ev:
        flush.zero_()          # L2 flush between timed iterations (outside the event pair)
        e0.record(stream)
        step()
        e1.record(stream)
    barrier()
    wall = time.perf_counter() - wall0
    launches = (snn.kernel_launches() - launches0) if not use_graph else \
        (1 if group is not None else len(layers)) * args.steps
    step_ms = [e0.elapsed_time(e1) for e0, e1 in ev]
    total_ms = float(sum(step_ms))

    # ---- check what was timed: outputs of the timed launches against the oracle (rank 0, after the timed region)
    checked = None
    if rank == 0 and not args.no_check:
        import oracle
        oracle.build()
        torch.cuda.synchronize(dev)
        checked = True
        picks = [(len(layers) - 1, nb)] + ([(0, min(2, nb))] if len(layers) > 1 else [])
        for j, n_img in picks:
            shape, p = workload.layers[j], params[j]
            a_np = host_acts[j][:n_img].numpy()
            if shape.ksize == 1:
                ref = (oracle.conv1x1_bin(p.codebook, workload.tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out,
                                          shape.stride, a_np.view(np.uint32))[1] if workload.act == "bin" else
                       oracle.conv1x1_f16(p.codebook, workload.tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out,
                                          shape.stride, a_np))
            elif workload.act == "bin":
                ref = oracle.conv_bin(p.codebook, workload.tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out,
                                      shape.stride, shape.pad, a_np.view(np.uint32))[1]
            else:
                ref = oracle.conv_f16(p.codebook, workload.tau, p.idx_packed, p.alpha, shape.c_in, shape.c_out,
                                      shape.stride, shape.pad, a_np)
            got = outs[j][:n_img].cpu().numpy()
            if workload.act == "bin":
                ok = bool((got == ref).all())
            else:
                sigma = p.alpha.astype(np.float64) * np.sqrt(float(shape.ksize ** 2 * shape.c_in))
                bound = 2e-2 * np.maximum(np.abs(ref.astype(np.float64)), sigma[None, None, None, :])
                ok = bool((np.abs(got.astype(np.float64) - ref) <= bound).all())
            checked = checked and ok

    # ---- the same step as one snn_conv_forward launch per layer, back to back on one stream
    k_side = max(3, min(30, args.steps))
    seq_ms = None
    if group is not None and not args.group_only:
        seq_graph = as_graph(lambda s: launch_layers(all_idx, s)) if use_graph else None
        seq_ms = timed(seq_graph.replay if use_graph else (lambda: launch_layers(all_idx, stream)), k_side)

    # ---- per-layer device time (L2 flushed before every layer)
    layer_ms = [0.0] * len(layers)
    if not args.group_only:
        reps = max(3, min(20, args.steps))
        for j in all_idx:
            gj = as_graph(lambda s, j=j: launch_layers([j], s)) if use_graph else None
            layer_ms[j] = timed(gj.replay if use_graph else (lambda j=j: launch_layers([j], stream)), reps, warm=1)

    # ---- the grouped step writing packed signs (1 bit per output) instead of fp32
    bits_ms = None
    if group is not None and workload.act == "bin":
        bit_outs = group.alloc_outs(snn.OUT_BITS)
        bits_ms = timed(lambda: group.forward(acts, bit_outs, snn.OUT_BITS, stream), k_side)
        del bit_outs

    # ---- the layers as a dependent chain through packed signs, ONE launch (snn_conv_stack_forward)
    stack_ms = None
    shapes = workload.layers
    chains = len(shapes) > 1 and all(a.c_out == b.c_in and a.h_out == b.h and a.w_out == b.w
                                     for a, b in zip(shapes, shapes[1:]))
    if workload.act == "bin" and chains and forced in (snn.PATH_AUTO, snn.PATH_DECODED_TC):
        stack = snn.SnnConvStack(layers, nb, shapes[0].h, shapes[0].w)
        s_out = stack.alloc_out(snn.OUT_F32)
        sg = as_graph(lambda s: stack.forward(acts[0], s_out, snn.OUT_F32, s)) if use_graph else None
        stack_ms = timed(sg.replay if use_graph else (lambda: stack.forward(acts[0], s_out, snn.OUT_F32, stream)), k_side)
        stack.destroy()
    clocks = sampler.stop()

    # ---- end to end through the host-buffer entry point: H2D of the inputs and D2H of the results inside the timing
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    for j, layer in enumerate(layers):
        layer.forward_host(host_acts[j], host_outs[j], snn.OUT_F32, paths[j])
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        for j, layer in enumerate(layers):
            layer.forward_host(host_acts[j], host_outs[j], snn.OUT_F32, paths[j])
    torch.cuda.synchronize(dev)
    e2e_ms = (time.perf_counter() - t0) / e2e_steps * 1e3
    h2d = sum(a.numel() * a.element_size() for a in host_acts)
    d2h = sum(o.numel() * o.element_size() for o in host_outs)

    # ---- measured ceilings of this device, by the library's own microbenchmarks
    store_gbs = snn.microbench(6, local_rank) / 1e9            # write-only stream of 16-byte stores
    mma_fp4 = snn.microbench(5, local_rank)                    # MAC/s, e2m1 MMAs of N = 240 as the kernel issues them
    mma_f16 = snn.microbench(7, local_rank)                    # MAC/s, fp16 MMAs of N = 256

    # max over ranks of the device-timed totals; every rank ran a batch of its own (weak scaling)
    total_ms, e2e_ms = replicas.max_over_ranks([total_ms, e2e_ms], world, dev)
    ms_per_step = total_ms / args.steps
    value = nb * world / (ms_per_step * 1e-3)
    e2e_value = nb * world / (e2e_ms * 1e-3)

    # ---- roofline of the dominant kernel (the path whose launches take the largest share of the step)
    by_path = {}
    for j, (shape, pth) in enumerate(zip(workload.layers, paths)):
        d = by_path.setdefault(pth, {"ms": 0.0, "macs": 0, "bytes": 0, "launches": 0})
        d["ms"] += layer_ms[j]
        d["macs"] += shape.dense_macs(nb)
        d["bytes"] += (shape.in_bytes_bin(nb) if workload.act == "bin" else shape.in_bytes_f16(nb)) + shape.out_bytes(nb)
        d["launches"] += 1
    dom = max(by_path, key=lambda k: by_path[k]["ms"])
    d = by_path[dom]
    sec = d["ms"] * 1e-3
    kernel_name = snn.PATH_NAMES[dom]
    if group is not None:
        # one kernel does the whole step: its launch duration is the step time measured in the timed region
        dom = snn.PATH_DECODED_TC
        d = {"ms": ms_per_step, "macs": workload.dense_macs(), "bytes": workload.algorithmic_bytes(), "launches": 1}
        sec = ms_per_step * 1e-3
        kernel_name = "tcg_conv_kernel (grouped decoded_tc)"
    elif len(by_path) == 1:
        # every launch of the step is this path's kernel, back to back: use the time of the timed region
        d = dict(d, ms=ms_per_step)
        sec = ms_per_step * 1e-3
    hbm_frac = d["bytes"] / sec / 1e9 / peaks["hbm_gbs"]
    extras = {}
    if dom == snn.PATH_DECODED_TC:
        # Dense contraction.  The kernel is timed alone (L2 flush between launches, clocks at their maximum), so
        # the burst figure applies.  Binary activations run on 4-bit e2m1 operands: measured bf16 x 4, the
        # nominal e2m1 : bf16 ratio; fp16 activations: x 1.
        ratio = 4.0 if workload.act == "bin" else 1.0
        peak = peaks["bf16_tflops"] * ratio
        achieved = 2 * d["macs"] / sec / 1e12
        pipe = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak}
        extras["peak_source"] = (peaks["source"] + (": bf16 burst x 4 nominal (e2m1 operands)" if workload.act == "bin"
                                                     else ": bf16 burst x 1 (fp16 operands)"))
        extras["frac_of_int8_peak"] = achieved / (peaks["bf16_tflops"] * 2.0) if workload.act == "bin" else None
        extras["mma_measured_tflops"] = 2 * (mma_fp4 if workload.act == "bin" else mma_f16) / 1e12
        extras["frac_of_mma_measured"] = achieved / extras["mma_measured_tflops"]
    elif dom == snn.PATH_DECODED:
        # one POPC per 32 MACs; 16 POPC lanes per SM per clock on 148 SMs at the maximum SM clock
        peak = 148 * 16 * peaks["sm_max_mhz"] * 1e6 / 1e12
        achieved = d["macs"] / 32 / sec / 1e12
        pipe = {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "Tpopc/s", "frac": achieved / peak}
        extras["popc_measured_per_s"] = snn.microbench(0, local_rank)
        extras["peak_source"] = "16 POPC lanes x 148 SMs x max SM clock"
    else:
        # one 4-pixel shared-memory word per (c_out, c_in, 4 pixels); 32 words per SM per clock
        peak = 148 * 32 * peaks["sm_max_mhz"] * 1e6 / 1e12
        achieved = d["macs"] / 9 / 4 / sec / 1e12
        pipe = {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "Tlds/s", "frac": achieved / peak}
        extras["lds_measured_per_s"] = snn.microbench(3, local_rank)
        extras["peak_source"] = "32 shared-memory words x 148 SMs x max SM clock"
    if hbm_frac >= pipe["frac"]:
        roofline = {"bound": "hbm", "achieved": d["bytes"] / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": hbm_frac}
        extras["hbm_peak_source"] = peaks["source"] + ": copy rate of MEASURED_PEAKS.json"
    else:
        roofline = pipe
    floor_ms = workload.algorithmic_bytes() / (peaks["hbm_gbs"] * 1e9) * 1e3
    roofline.update({"traffic": _profiled_traffic(kernel_name, nb, workload), "kernel": kernel_name,
                     "launches_per_step": d["launches"],
                     "share_of_step": 1.0 if group is not None else d["ms"] / max(sum(layer_ms), 1e-9),
                     "algorithmic_bytes_per_launch": d["bytes"] / d["launches"],
                     "algorithmic_ops_per_launch": 2 * d["macs"] / d["launches"],
                     "hbm_frac": hbm_frac, "pipe_frac": pipe["frac"],
                     "store_stream_gbs": store_gbs,
                     "frac_of_store_stream": d["bytes"] / sec / 1e9 / store_gbs,
                     # the same step as one launch per layer, against the same floor
                     "per_layer_launches_ms": seq_ms,
                     "per_layer_launches_frac": None if seq_ms is None else floor_ms / seq_ms,
                     **extras})

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        # the type the dominant path computes in: e2m1 operands (+/-1 and 0, exact) with fp32 accumulation on the
        # tensor cores, fp16 operands in the fp16-activation variant, int32 on the ALU paths
        "dtype": ("f16" if workload.act != "bin" else "e2m1" if dom == snn.PATH_DECODED_TC else "int32"),
        "data": "synthetic",
        "config": {"workload": _workload_name(workload), "layers": len(layers), "batch_per_gpu": nb,
                   "tau": workload.tau, "index_skew": args.index_skew,
                   "l2": "flushed between timed steps (256 MB write)",
                   "launch": ("one grouped launch of all layers (snn_conv_group_forward), " if group is not None else "") +
                             ("host calls" if args.no_graph else
                              "replayed as a CUDA graph" if group is not None else
                              "CUDA graph of the per-layer C-ABI launches"),
                   "grouped": group is not None,
                   "paths": [snn.PATH_NAMES[p] for p in paths]},
        "checked": checked,
        "effective_tops": 2 * workload.dense_macs() * world / (ms_per_step * 1e-3) / 1e12,
        "hbm_floor_ms_per_step": floor_ms,
        "step_frac_of_hbm_floor": floor_ms / ms_per_step,
        "layer_ms": [round(v, 5) for v in layer_ms],
        "per_layer_launches": None if seq_ms is None else {
            "ms_per_step": seq_ms, "value": nb / (seq_ms * 1e-3), "unit": UNIT + " per GPU",
            "what": "the same step as one snn_conv_forward launch per layer, back to back on one stream"},
        "packed_sign_outputs": None if bits_ms is None else {
            "ms_per_step": bits_ms, "value": nb / (bits_ms * 1e-3), "unit": UNIT + " per GPU",
            "what": "the grouped step with SNN_OUT_BITS (signs of the outputs packed as the next layer's input) "
                    "instead of fp32 outputs; host launches, not a graph"},
        "dependent_stack": None if stack_ms is None else {
            "ms_per_step": stack_ms, "value": nb / (stack_ms * 1e-3), "unit": UNIT + " per GPU",
            "what": "the layers as a dependent chain in ONE launch (snn_conv_stack_forward): every layer's packed "
                    "thresholded signs are the next layer's input, the last layer writes fp32"},
        "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "wall_s_timed_region": wall,
    }

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        n_img = oracle_sample_images(workload, 15.0)
        t_or, passes = 0.0, 0
        while t_or < 10.0 and passes < 8:   # about 10-30 s of CPU work in all
            t_or += time_oracle_stack(workload, n_img)
            passes += 1
        line["cpu_baseline"] = {
            "value": n_img * passes / t_or, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{n_img} of {nb} images through all {len(layers)} layers, {passes} passes, {t_or:.1f} s",
        }
    elif rank == 0:
        line["cpu_baseline"] = None
    if rank == 0:
        print(json.dumps(line), flush=True)
    if group is not None:
        group.destroy()
    for layer in layers:
        layer.destroy()
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18", choices=list(wl.WORKLOAD_NAMES))
    ap.add_argument("--tau", type=int, default=None)
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--path", default="auto", choices=["auto", "reuse", "decoded", "decoded_tc"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--index-skew", default="none", choices=["none", "deep", "top64"],
                    help="draw the indices from the kernel-frequency profile of trained layers (Sec. 4.2) "
                         "instead of uniformly")
    ap.add_argument("--no-check", action="store_true", help="skip the oracle check of the timed outputs")
    ap.add_argument("--group-only", action="store_true",
                    help="time only the grouped launch: no tuning, no per-layer timings (profiling aid)")
    ap.add_argument("--per-layer", action="store_true",
                    help="run the step as one launch per layer instead of one grouped launch of all layers")
    ap.add_argument("--no-graph", action="store_true", help="launch every layer from the host instead of a CUDA graph")
    ap.add_argument("--layers", default=None, help="a:b restricts the stack to layers [a, b) (profiling aid)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
