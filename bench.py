#!/usr/bin/env python
"""Benchmark of the dual-routed MWQ MoE layer (one step = one pass of the whole hot path over one batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload mixtral_decode] [--tokens 64] [--path auto|cuda_core|tensor]
                    [--min-region-s 1.0] [--others all|layers|none]

Prints ONE JSON line.  The timed region is exactly K steps between a barrier + synchronize on both sides;
it is repeated until --min-region-s seconds of device time are timed and the median region gives `value`
(uninstrumented steps; the per-stage times behind `roofline` come from a separate pass).  With the default
workload on one GPU the line also carries short legs of the other benchmark configurations
(`other_workloads`: decode batches of 1, 8 and 32 tokens, the 2048-token prefill batch, the fine-grained
layer, the 32-layer stack).  N > 1 runs independent replicas, one process per GPU, no data-path collective;
the barrier and the max-over-ranks timing use NCCL; started as a plain script with --gpus N it starts the
N ranks itself.  `--impl reference` times the CPU oracle on the host cores on a bounded sample of the same
workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2504_15299_b200 import synth  # noqa: E402

METRIC = "moe_layer_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, each from one ncu capture of
# the same workload through this script (the summaries of those captures are committed beside the numbers
# they come from); key = workload:tokens:stage:path
NCU_TRAFFIC = {"mixtral_decode:T64:gate_up:auto": 1042948288, "mixtral_decode:T64:down:auto": 536264624,
               "mixtral_prefill:T2048:gate_up:auto": 1649747408, "mixtral_prefill:T2048:down:auto": 1008871152,
               "finegrained:T256:gate_up:auto": 462040064, "finegrained:T256:down:auto": 234176768}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------------
# algorithmic bytes: what the method has to read at the routed widths - per active expert and matrix the
# packed prefix up to the widest width routed to that expert in this call, read once, plus activations
# in and outputs out
# ------------------------------------------------------------------------------------------------
def matrix_bytes(rows, cols, g, bits_read, scale_steps=0):
    """codes at the width read + (fp16 scale, fp16 offset) per row and group (+ one fp16 scale per extra bit read
    when the residual scales are free)."""
    return rows * cols * bits_read // 8 + rows * (cols // g) * (4 + 2 * scale_steps)


def algorithmic_bytes(wl, T, group_off, scale_mode=0):
    """Bytes per layer call from the realised routing: every plane of an active expert up to the
    largest width routed to it is read once; plus activations in/out and the h round trip."""
    K = len(wl.bits)
    hist = [group_off[i + 1] - group_off[i] for i in range(wl.n_experts * K)]
    gu = dn = 0
    active = 0
    for e in range(wl.n_experts + wl.n_shared):
        if e < wl.n_experts:
            ks = [kk for kk in range(K) if hist[e * K + kk] > 0]
            if not ks:
                continue
            b = wl.bits[max(ks)]
        else:
            b = wl.bits[-1]
        active += 1
        steps = b - wl.bits[0] if scale_mode == 1 else 0
        gu += 2 * matrix_bytes(wl.d_ffn, wl.d_model, wl.group_size, b, steps)
        dn += matrix_bytes(wl.d_model, wl.d_ffn, wl.group_size, b, steps)
    A_tot = T * (wl.top_k + wl.n_shared)
    io_gu = A_tot * wl.d_model * 2 + A_tot * wl.d_ffn * 2       # gathered x in, h out (16-bit)
    io_dn = A_tot * wl.d_ffn * 2 + A_tot * wl.d_model * 4       # h in, expert outputs out (fp32)
    io_layer = 2 * T * wl.d_model * 2 + T * wl.top_k * 17
    return {"gate_up": gu + io_gu, "down": dn + io_dn, "layer": gu + dn + io_layer, "active_experts": active}


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """Polls NVML (read-only queries) from a background thread every ~2 ms while the timed region runs:
    SM clock, max SM clock and the active clock-event (throttle) reasons."""

    REASONS = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
               "sw_thermal_slowdown": 0x20, "hw_power_brake_slowdown": 0x80}

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.samples = []
        self.reason_bits = 0
        self.max_mhz = None
        self._stop = None
        self._thread = None
        self._nvml = None

    def start(self):
        try:
            import threading

            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            # CUDA_VISIBLE_DEVICES may renumber devices: match by PCI bus id
            bus = torch.cuda.get_device_properties(self.gpu).pci_bus_id if hasattr(
                torch.cuda.get_device_properties(self.gpu), "pci_bus_id") else None
            handle = None
            if bus is not None:
                for i in range(pynvml.nvmlDeviceGetCount()):
                    h = pynvml.nvmlDeviceGetHandleByIndex(i)
                    if pynvml.nvmlDeviceGetPciInfo(h).bus == bus:
                        handle = h
                        break
            if handle is None:
                handle = pynvml.nvmlDeviceGetHandleByIndex(self.gpu)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
            self._stop = threading.Event()

            def poll():
                while not self._stop.is_set():
                    try:
                        self.samples.append(float(pynvml.nvmlDeviceGetClockInfo(handle, pynvml.NVML_CLOCK_SM)))
                        self.reason_bits |= int(pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(handle))
                    except Exception:
                        pass
                    time.sleep(0.002)

            self._thread = threading.Thread(target=poll, daemon=True)
            self._thread.start()
        except Exception:
            self._thread = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": []}
        if self._thread is None:
            return out
        self._stop.set()
        self._thread.join(timeout=2)
        if self.samples:
            sm = sorted(self.samples)
            out["sm_mhz"] = sm[len(sm) // 2]
            out["samples"] = len(sm)
        out["reasons"] = sorted(n for n, bit in self.REASONS.items() if self.reason_bits & bit)
        return out


# ------------------------------------------------------------------------------------------------
# oracle legs (CPU)
# ------------------------------------------------------------------------------------------------
class OracleSample:
    """The oracle on a bounded sample: the first `n_tok` tokens of the batch through routing,
    dequantization at the routed widths, the expert FFN restricted to the first `n_hidden_groups`
    groups of hidden units (the FFN cost is linear in the hidden units: each contributes one term
    of the down projection), and the combine.  Time is scaled by F / hidden units used."""

    def __init__(self, wl, T, n_tok, n_hidden_groups, device_for_inputs="cpu"):
        import numpy as np
        from oracle import mwq, routing
        self.np, self.mwq, self.routing = np, mwq, routing
        self.wl, self.T, self.n_tok = wl, T, n_tok
        g = wl.group_size
        self.hid = min(wl.d_ffn, n_hidden_groups * g)
        x = synth.tokens_bf16(wl, T, device_for_inputs)
        self.x = x.to("cpu", torch.float32).numpy()
        self.gw = synth.gate_weight_bf16(wl, "cpu").to(torch.float32).numpy()
        self.fb = synth.forced_bit_idx(wl, T, "cpu").numpy()
        rt = routing.route(self.x, E=wl.n_experts, K=len(wl.bits), top_k=wl.top_k,
                           renormalize=bool(wl.renormalize), gate_w=self.gw, forced_bit_idx=self.fb)
        experts = sorted({int(e) for t in range(n_tok) for e in rt.topk_idx[t]}) + \
            [wl.n_experts + s for s in range(wl.n_shared)]
        sub = torch.arange(self.hid)
        self.packed = {}
        for e in experts:          # setup (offline quantization), not timed
            Wg = synth.expert_matrix(wl, e, 0, device_for_inputs, rows=sub).cpu().numpy()
            Wu = synth.expert_matrix(wl, e, 1, device_for_inputs, rows=sub).cpu().numpy()
            # columns 0..hid-1 of the [d, F] down projection (whole groups along F)
            Wd = synth.expert_matrix(wl, e, 2, device_for_inputs, cols=sub).cpu().numpy()
            self.packed[e] = tuple(mwq.quantize(W, wl.bits, g) for W in (Wg, Wu, Wd))

    def step(self):
        """One timed pass; returns (seconds, scale factor to the full FFN)."""
        from oracle import moe
        wl = self.wl
        t0 = time.perf_counter()
        rt = self.routing.route(self.x, E=wl.n_experts, K=len(wl.bits), top_k=wl.top_k,
                                renormalize=bool(wl.renormalize), gate_w=self.gw, forced_bit_idx=self.fb)
        moe.moe_layer(self.x, rt, lambda e: self.packed[e], wl.bits, wl.n_experts, wl.n_shared,
                      tokens=range(self.n_tok))
        dt = time.perf_counter() - t0
        return dt, wl.d_ffn / self.hid


def oracle_tokens_per_s(wl, T, n_tok, n_hidden_groups, steps, warmup, device_for_inputs="cpu"):
    s = OracleSample(wl, T, n_tok, n_hidden_groups, device_for_inputs)
    for _ in range(warmup):
        s.step()
    tot = 0.0
    for _ in range(max(steps, 1)):
        dt, scale = s.step()
        tot += dt * scale
    per_step = tot / max(steps, 1)
    return n_tok / per_step, per_step, s.hid


def used_threads():
    try:
        import threadpoolctl
        n = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] or [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = synth.WORKLOADS[args.workload]
    T = args.tokens or synth.WORKLOADS[args.workload].tokens[-1]
    total_steps = args.steps + args.warmup
    # size the sample so the whole run stays within ~2.5 minutes: calibrate on one hidden group
    t0 = time.perf_counter()
    v, per, _ = oracle_tokens_per_s(wl, T, 1, 1, 1, 0)
    calib = time.perf_counter() - t0
    groups = 1
    budget = 150.0 / max(total_steps, 1)
    while groups < 8 and calib * groups * 2 < budget * 0.5:
        groups *= 2
    value, per_step, hid = oracle_tokens_per_s(wl, T, 1, groups, args.steps, args.warmup)
    cores = used_threads()
    sample = (f"first token of the T={T} batch, all its experts at the routed widths, hidden units "
              f"0..{hid - 1} of {wl.d_ffn} per expert, time scaled by {wl.d_ffn}/{hid} (extrapolated)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(wl, T, "cpu oracle"),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def max_over_ranks(ms: float, dist, device) -> float:
    """Step time of the job = the slowest rank's device time."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput of `world` independent replicas (weak scaling: fixed tokens per rank)."""
    return tokens_per_rank * world / (ms_per_step * 1e-3)


# ------------------------------------------------------------------------------------------------
# timing helpers
# ------------------------------------------------------------------------------------------------
L2_BYTES = 126 * 1024 * 1024


def _sync_all(dist):
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
        torch.cuda.synchronize()


def time_regions(run_region, steps, dist, dev, min_region_s, max_regions=200):
    """Times regions of exactly `steps` steps each (barrier + synchronize on both sides, device time, max over
    ranks) until `min_region_s` seconds of device time have been timed.  run_region(r) enqueues one region's steps
    and returns its device milliseconds (it may time every step by itself, see LayerBench).  Returns the list of
    per-region milliseconds; every rank takes the same number of regions (the decision uses the reduced time)."""
    out = []
    total = 0.0
    for r in range(max_regions):
        _sync_all(dist)
        ms = max_over_ranks(run_region(r), dist, dev)
        out.append(ms)
        total += ms
        if total >= min_region_s * 1e3:
            break
    return out


def median(v):
    s = sorted(v)
    n = len(s)
    return s[n // 2] if n % 2 else 0.5 * (s[n // 2 - 1] + s[n // 2])


class LayerBench:
    """One single-layer workload on this rank's GPU: packed experts, four rotating token batches (inputs
    resident in HBM), the workspace, and the algorithmic bytes of every batch from its realised routing."""

    N_BATCHES = 4

    def __init__(self, B, wl, T, path_name, dev, rank=0, blobs=None, scale_mode=0):
        self.B, self.wl, self.T, self.dev, self.path_name, self.scale_mode = B, wl, T, dev, path_name, scale_mode
        path = {"auto": B.PATH_AUTO, "cuda_core": B.PATH_CUDA_CORE, "tensor": B.PATH_TENSOR}[path_name]
        self.cfg = B.Config.from_workload(wl, kernel_path=path, scale_mode=scale_mode)
        if blobs is None:
            blobs = []
            for e in range(wl.n_experts + wl.n_shared):
                for m in range(3):
                    W = synth.expert_matrix(wl, e, m, device=dev)
                    blobs.append(B.pack_mwq(self.cfg, W))
                    del W
        self.blobs = blobs
        self.gw = synth.gate_weight_bf16(wl, dev)
        nb = self.N_BATCHES
        self.xs = [synth.tokens_bf16(wl, T, dev, step=rank * 100 + i) for i in range(nb)]
        self.fbs = [synth.categorical(wl.seed + rank * 100 + i, synth.TID_FORCED_BITS, (T, wl.top_k), wl.bit_probs, dev)
                    for i in range(nb)]
        self.logits = [synth.zipf_logits(wl, T, dev) for _ in range(nb)] if wl.zipf_logits else None
        self.ws = torch.empty(B.workspace_bytes(self.cfg, T), dtype=torch.uint8, device=dev)
        self.y = torch.empty_like(self.xs[0])
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.alg = []
        for i in range(nb):
            r = B.route(self.cfg, self.xs[i], workspace=self.ws, **self.kw(i))
            torch.cuda.synchronize()
            self.alg.append(algorithmic_bytes(wl, T, r.group_off.cpu().tolist(), scale_mode))
        self.layer_bytes = sum(a["layer"] for a in self.alg) / nb
        # a step that streams less than a few L2 sizes could be served partly from L2 by the step before it:
        # such workloads are timed step by step with an L2 flush (a 256 MiB write) between the steps
        self.flush = self.layer_bytes < 4 * L2_BYTES
        self.flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev) if self.flush else None
        self.decode = -(-T * wl.top_k // wl.n_experts) <= 40 and scale_mode == 0

    def kw(self, i, fb=None):
        d = {"forced_bit_idx": self.fbs[i] if fb is None else fb}
        if self.logits is not None:
            d["logits"] = self.logits[i]
        else:
            d["gate_w"] = self.gw
        return d

    def step(self, i, events=None):
        j = i % self.N_BATCHES
        self.B.moe_forward(self.cfg, self.xs[j], self.blobs, y=self.y, workspace=self.ws, device_status=self.status,
                           stage_events=events, **self.kw(j))

    def region(self, steps, first=0):
        """Enqueues `steps` uninstrumented steps and returns their device time in ms (waits for them)."""
        stream = torch.cuda.current_stream()
        if not self.flush:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(steps):
                self.step(first + i)
            e1.record(stream)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(steps):
            self.flush_buf.zero_()
            evs[i][0].record(stream)
            self.step(first + i)
            evs[i][1].record(stream)
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in evs)

    def stage_pass(self, steps):
        """A separate, instrumented pass: the library records events around its stages on every step."""
        B = self.B
        stream = torch.cuda.current_stream()
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(B.N_STAGES + 1)] for _ in range(steps)]
        for row in evs:
            for ev in row:
                ev.record(stream)                      # creates the handle
        torch.cuda.synchronize()
        for i in range(steps):
            if self.flush:
                self.flush_buf.zero_()
            self.step(i, evs[i])
        torch.cuda.synchronize()
        stage_ms = [sum(evs[i][s].elapsed_time(evs[i][s + 1]) for i in range(steps)) / steps for s in range(B.N_STAGES)]
        used = [self.alg[i % self.N_BATCHES] for i in range(steps)]
        return stage_ms, used

    def roofline(self, stage_ms, used, ms_per_step, clocks=None):
        """Roofline of the stage with the largest device time, and of the whole layer call."""
        B, wl, T = self.B, self.wl, self.T
        names = B.STAGE_NAMES
        dom = max(range(B.N_STAGES), key=lambda s: stage_ms[s])
        dom_name = names[dom]
        peak, peak_kind = measured_peaks()
        dom_bytes = sum(u.get(dom_name, u["layer"]) for u in used) / len(used)
        layer_bytes = sum(u["layer"] for u in used) / len(used)
        achieved = dom_bytes / (stage_ms[dom] * 1e-3) / 1e9
        rf = {"bound": "hbm", "kernel": dom_name, "achieved": achieved, "peak": peak, "unit": "GB/s",
              "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
              "traffic": NCU_TRAFFIC.get(f"{wl.name}:T{T}:{dom_name}:{self.path_name}"),
              "algorithmic_bytes_per_launch": dom_bytes,
              "stage_ms": dict(zip(names, stage_ms)), "stage_samples": len(used),
              "layer": {"algorithmic_bytes": layer_bytes,
                        "achieved_gbs": layer_bytes / (ms_per_step * 1e-3) / 1e9,
                        "frac": layer_bytes / (ms_per_step * 1e-3) / 1e9 / peak}}
        dtype = "f32" if self.path_name == "cuda_core" else "i8"
        small_load = -(-T * wl.top_k // wl.n_experts) <= 40       # decode-sized: bound by the bytes whichever kernel runs
        if self.scale_mode == 1 and small_load and self.path_name != "cuda_core":
            dtype = "f16"
        if not self.decode and not small_load and self.path_name != "cuda_core":
            # prefill-sized expert loads (the grouped dequant-GEMM) are bound by the tensor cores: the dominant
            # kernel against the measured dense 16-bit matmul rates (fp16 operands have the nominal rate of the
            # bf16 the peaks were measured with); both the burst and the sustained (power-capped) figure
            dtype = "f16"
            A_tot = T * (wl.top_k + wl.n_shared)
            flops = {"gate_up": A_tot * 2 * 2 * wl.d_model * wl.d_ffn, "down": A_tot * 2 * wl.d_model * wl.d_ffn}
            burst, sustained, tkind = measured_tensor_peaks()
            tf = flops.get(dom_name, sum(flops.values())) / (stage_ms[dom] * 1e-3) / 1e12
            # a run short enough to stay at full clocks is compared with the burst figure, one that sits at the
            # power cap with the sustained one
            capped = bool(clocks and "sw_power_cap" in (clocks.get("reasons") or []))
            tpeak = sustained if capped else burst
            rf.update({"bound": "tensor", "achieved": tf, "peak": tpeak, "unit": "TFLOP/s", "frac": tf / tpeak,
                       "peak_kind": f"of {tkind} ({'sustained: run at the power cap' if capped else 'burst: run at full clocks'})",
                       "frac_of_burst": tf / burst, "frac_of_sustained": tf / sustained,
                       "algorithmic_flops_per_launch": flops.get(dom_name)})
            lt = sum(flops.values()) / (ms_per_step * 1e-3) / 1e12
            rf["layer"] = {"algorithmic_flops": sum(flops.values()), "achieved_tflops": lt, "frac": lt / tpeak}
        return rf, dtype

    def l2_note(self):
        if self.flush:
            return ("L2 flushed between steps: a 256 MiB buffer is written before every step (a step streams "
                    f"{self.layer_bytes / 1e6:.0f} MB, less than four L2 sizes) and every step is timed by its own events")
        return (f"inputs larger than L2: each step streams the routed planes of every active expert "
                f"({self.layer_bytes / 1e6:.0f} MB per layer call against a 126 MB L2); four token batches are rotated")


def measured_tensor_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured"
        except Exception:
            pass
    return 1590.0, 1400.0, "fallback"


def workload_config(wl, T, path, l2=None):
    return {"workload": f"{wl.name} T={T}: d={wl.d_model} ffn={wl.d_ffn} E={wl.n_experts} top{wl.top_k} "
                        f"g={wl.group_size} bits={list(wl.bits)} p={list(wl.bit_probs)}"
                        + (f" +{wl.n_shared} shared" if wl.n_shared else ""),
            "tokens_per_step": T, "kernel_path": path, "l2": l2 or "inputs larger than L2"}


def short_leg(B, wl, T, dev, blobs=None, steps=20, min_s=0.25, scale_mode=0):
    """A short device-timed leg of another configuration (same rules: warm-up, regions of `steps` steps,
    clocks sampled during the regions, stages from a separate pass)."""
    lb = LayerBench(B, wl, T, "auto", dev, blobs=blobs, scale_mode=scale_mode)
    for i in range(3):
        lb.step(i)
    torch.cuda.synchronize()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    regions = time_regions(lambda r: lb.region(steps, r * steps), steps, None, dev, min_s)
    clocks = sampler.stop()
    assert int(lb.status.item()) == 0, f"device status {int(lb.status.item())}"
    ms = median(regions) / steps
    stage_ms, used = lb.stage_pass(8)
    rf, dtype = lb.roofline(stage_ms, used, ms, clocks)
    return {"workload": workload_config(wl, T, "auto", lb.l2_note())["workload"]
                        + (" free per-step residual scales (scale_mode 1)" if scale_mode else ""),
            "blobs": lb.blobs, "tokens_per_step": T,
            "ms_per_step": ms, "tokens_per_s": T / (ms * 1e-3), "dtype": dtype, "regions": len(regions),
            "timed_region_s": sum(regions) * 1e-3, "l2": lb.l2_note(), "clocks": clocks, "roofline": rf}


# ------------------------------------------------------------------------------------------------
# layer stack (the 32-layer decode configuration): one step = every layer once, replayed as a CUDA graph
# ------------------------------------------------------------------------------------------------
def stack_bench(B, wl, T, L, dev, steps, warmup, use_graph=True, min_s=1.0, e2e=True):
    cfg = B.Config.from_workload(wl)
    layers = []
    for l in range(L):
        blobs = []
        for e in range(wl.n_experts + wl.n_shared):
            for m in range(3):
                W = synth.expert_matrix(wl, e, m, device=dev, layer=l)
                blobs.append(B.pack_mwq(cfg, W))
                del W
        layers.append((blobs, synth.gate_weight_bf16(wl, dev, layer=l), synth.bit_router_weight_bf16(wl, dev, layer=l)))
    ws = torch.empty(B.workspace_bytes(cfg, T), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    n_batches = 4
    xs = [synth.tokens_bf16(wl, T, dev, step=1000 + i) for i in range(n_batches)]
    x = torch.empty_like(xs[0])
    xn = torch.empty_like(x)

    def one_step():
        for blobs, gw, bw in layers:
            B.stack_layer(cfg, x, xn, blobs, gate_w=gw, bit_w=bw, workspace=ws, device_status=status)

    # algorithmic bytes of a step from the realised routing of every layer (batch 0, eager pass)
    x.copy_(xs[0])
    step_bytes = 0
    for blobs, gw, bw in layers:
        B.stack_layer(cfg, x, xn, blobs, gate_w=gw, bit_w=bw, workspace=ws, device_status=status)
        r = B.route(cfg, xn, gate_w=gw, bit_w=bw)
        torch.cuda.synchronize()
        step_bytes += algorithmic_bytes(wl, T, r.group_off.cpu().tolist())["layer"]

    side = torch.cuda.Stream()
    graph = None
    if use_graph:
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            one_step()                     # warm-up on the capture stream (function attributes, tensor maps)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            one_step()

    def step(i):
        x.copy_(xs[i % n_batches])
        if graph is not None:
            graph.replay()
        else:
            one_step()

    for i in range(max(warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()

    def region(r):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            step(r * steps + i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    regions = time_regions(region, steps, None, dev, min_s)
    clocks = sampler.stop()
    ms_per_step = median(regions) / steps
    assert int(status.item()) == 0, f"device status {int(status.item())}"

    e2e_out = None
    if e2e:
        # end to end: tokens from pinned host memory, the stack, result back to the host, every step
        hx = [t.cpu().pin_memory() for t in xs]
        hy = torch.empty_like(hx[0]).pin_memory()

        def e2e_step(i):
            x.copy_(hx[i % n_batches], non_blocking=True)
            if graph is not None:
                graph.replay()
            else:
                one_step()
            hy.copy_(x, non_blocking=True)

        for i in range(3):
            e2e_step(i)
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for i in range(steps):
            e2e_step(i)
        f1.record()
        torch.cuda.synchronize()
        e2e_ms = f0.elapsed_time(f1) / steps
        e2e_out = {"value": T / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": hx[0].numel() * 2,
                   "d2h_bytes_per_step": hy.numel() * 2}

    peak, peak_kind = measured_peaks()
    achieved = step_bytes / (ms_per_step * 1e-3) / 1e9
    return {"ms_per_step": ms_per_step, "tokens_per_s": T / (ms_per_step * 1e-3), "regions": regions,
            "clocks": clocks, "e2e": e2e_out, "graph": graph is not None, "step_bytes": step_bytes,
            "launches_per_step": (B.forward_launch_count(cfg, T) + 1) * L,
            "roofline": {"bound": "hbm", "kernel": "whole step", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": None,
                         "algorithmic_bytes_per_step": step_bytes},
            "workload": f"{wl.name}: {L} layers of d={wl.d_model} ffn={wl.d_ffn} E={wl.n_experts} "
                        f"top{wl.top_k} g={wl.group_size} bits={list(wl.bits)}, widths from the per-expert "
                        f"bit-width routers, RMSNorm + residual per layer",
            "l2": f"inputs larger than L2: {L} layers of distinct packed experts ({step_bytes / 1e9:.1f} GB read per step)"}


def run_stack(args):
    from paper_2504_15299_b200 import binding as B, build
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    build.build_library()
    B.lib()
    wl = synth.WORKLOADS[args.workload]
    T = args.tokens or wl.tokens[-1]
    L = args.layers or wl.n_layers
    r = stack_bench(B, wl, T, L, dev, args.steps, args.warmup, use_graph=not args.no_graph, min_s=args.min_region_s)
    n_reg = len(r["regions"])
    line = {"metric": METRIC, "value": r["tokens_per_s"], "unit": UNIT, "n_gpus": 1, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "i8", "data": "synthetic",
            "config": {"workload": r["workload"], "tokens_per_step": T, "layers": L, "cuda_graph": r["graph"], "l2": r["l2"]},
            "timing": timing_block(r["regions"], args.steps),
            "clocks": r["clocks"], "e2e": r["e2e"],
            "gpu_launches": r["launches_per_step"] * args.steps * n_reg,
            "roofline": r["roofline"], "cpu_baseline": None}
    print(json.dumps(line))


def timing_block(regions, steps):
    per = [ms / steps for ms in regions]
    return {"regions": len(regions), "steps_per_region": steps, "timed_region_s": sum(regions) * 1e-3,
            "ms_per_step_median": median(per), "ms_per_step_min": min(per), "ms_per_step_max": max(per),
            "note": "each region is exactly `steps` steps between a barrier + synchronize on both sides; regions are "
                    "repeated until at least --min-region-s seconds of device time are timed; value uses the median region"}


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
def run_ours(args):
    from paper_2504_15299_b200 import binding as B, build
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build_library()
    if dist:
        dist.barrier()
    B.lib()

    wl = synth.WORKLOADS[args.workload]
    T = args.tokens or synth.WORKLOADS[args.workload].tokens[-1]
    lb = LayerBench(B, wl, T, args.path, dev, rank=rank, scale_mode=args.scale_mode)
    stream = torch.cuda.current_stream()

    for i in range(args.warmup):
        lb.step(i)
    _sync_all(dist)

    # ---- timed regions: K uninstrumented steps each, device time, max over ranks ----
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    regions = time_regions(lambda r: lb.region(args.steps, r * args.steps), args.steps, dist, dev, args.min_region_s)
    _sync_all(dist)
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step = median(regions) / args.steps
    assert int(lb.status.item()) == 0, f"device status {int(lb.status.item())}"

    # ---- per-stage device times: a separate pass with the library's stage events on every step ----
    stage_ms, used = lb.stage_pass(min(max(args.steps, 8), 40))

    # ---- end to end: pinned host inputs -> device, layer, result back to the host, every step ----
    # The serving loop a user of the library would write: two sets of device buffers, the copies on streams of
    # their own, so that the copy-in of step i + 1 and the copy-out of step i - 1 overlap the layer call of
    # step i.  Every step's inputs come from pinned host memory and every step's result lands in pinned host
    # memory inside the timed region; the region ends when the last result has arrived.
    nb = lb.N_BATCHES
    hx = [x.cpu().pin_memory() for x in lb.xs]
    hfb = [f.cpu().pin_memory() for f in lb.fbs]
    hy = [torch.empty_like(hx[0]).pin_memory() for _ in range(2)]
    dx = [torch.empty_like(lb.xs[0]) for _ in range(2)]
    dfb = [torch.empty_like(lb.fbs[0]) for _ in range(2)]
    dy = [torch.empty_like(lb.y) for _ in range(2)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]       # inputs of the buffer set have arrived
    ev_done = [torch.cuda.Event() for _ in range(2)]     # the layer call on the buffer set has finished
    ev_out = [torch.cuda.Event() for _ in range(2)]      # its result has left the device
    for b in range(2):
        ev_done[b].record(stream)
        ev_out[b].record(stream)

    def e2e_step(i):
        j, b = i % nb, i & 1
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_done[b])                   # the call two steps back has read these inputs
            dx[b].copy_(hx[j], non_blocking=True)
            dfb[b].copy_(hfb[j], non_blocking=True)
            ev_in[b].record(s_in)
        stream.wait_event(ev_in[b])
        stream.wait_event(ev_out[b])                      # the result two steps back has been copied out
        B.moe_forward(lb.cfg, dx[b], lb.blobs, y=dy[b], workspace=lb.ws, device_status=lb.status, **lb.kw(j, dfb[b]))
        ev_done[b].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[b])
            hy[b].copy_(dy[b], non_blocking=True)
            ev_out[b].record(s_out)

    for i in range(args.warmup):
        e2e_step(i)
    _sync_all(dist)

    def e2e_region(r):
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        for i in range(args.steps):
            e2e_step(args.warmup + r * args.steps + i)
        stream.wait_event(ev_out[0])
        stream.wait_event(ev_out[1])
        f1.record(stream)
        torch.cuda.synchronize()
        return f0.elapsed_time(f1)

    e2e_regions = time_regions(e2e_region, args.steps, dist, dev, min(args.min_region_s, 0.5))
    _sync_all(dist)
    e2e_ms = median(e2e_regions) / args.steps

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    roofline, dtype = lb.roofline(stage_ms, used, ms_per_step, clocks)
    lb_l2 = lb.l2_note()

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        v, per, hid = oracle_tokens_per_s(wl, T, 1, 32, 2, 0, device_for_inputs=dev)
        cpu = {"value": v, "unit": UNIT, "cores": used_threads(), "kind": "oracle",
               "sample": f"first token of the batch, all its experts at the routed widths, hidden units "
                         f"0..{hid - 1} of {wl.d_ffn} per expert, time scaled by {wl.d_ffn}/{hid} "
                         f"(extrapolated); 2 passes"}

    # ---- the other configurations, short legs in the same invocation (one GPU only) ----
    others = None
    if world == 1 and args.others and args.workload == "mixtral_decode" and args.path == "auto" and args.scale_mode == 0:
        others = []
        for t in wl.tokens:
            if t != T:
                others.append(short_leg(B, wl, t, dev, blobs=lb.blobs))
        wlp = synth.WORKLOADS["mixtral_prefill"]          # same seed and shapes: the same packed experts
        others.append(short_leg(B, wlp, wlp.tokens[-1], dev, blobs=lb.blobs, steps=10))
        wlf = synth.WORKLOADS["finegrained"]
        others.append(short_leg(B, wlf, wlf.tokens[-1], dev))
        # the same Mixtral-shaped layer with free per-step residual scales (Eq. 4 / Eq. 5): repacked, both batch sizes
        leg = short_leg(B, wl, T, dev, scale_mode=1)
        others.append(leg)
        others.append(short_leg(B, wlp, wlp.tokens[-1], dev, blobs=leg["blobs"], steps=10, scale_mode=1))
        for o in others:
            o.pop("blobs", None)
        torch.cuda.empty_cache()
        if args.others == "all":
            wls = synth.WORKLOADS["mixtral_stack"]
            r = stack_bench(B, wls, wls.tokens[-1], wls.n_layers, dev, 10, 3, use_graph=True, min_s=0.5, e2e=False)
            others.append({"workload": r["workload"], "tokens_per_step": wls.tokens[-1], "ms_per_step": r["ms_per_step"],
                           "tokens_per_s": r["tokens_per_s"], "dtype": "i8", "regions": len(r["regions"]),
                           "timed_region_s": sum(r["regions"]) * 1e-3, "l2": r["l2"], "clocks": r["clocks"],
                           "cuda_graph": r["graph"], "roofline": r["roofline"]})

    cfg_T = B.Config.from_workload(wl, scale_mode=args.scale_mode)
    line = {"metric": METRIC, "value": job_tokens_per_s(T, world, ms_per_step), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": dtype,
            "data": "synthetic", "config": workload_config(wl, T, args.path, lb_l2),
            "timing": timing_block(regions, args.steps),
            "clocks": clocks,
            "e2e": {"value": job_tokens_per_s(T, world, e2e_ms), "unit": UNIT,
                    "h2d_bytes_per_step": hx[0].numel() * 2 + hfb[0].numel(),
                    "d2h_bytes_per_step": hy[0].numel() * 2, "regions": len(e2e_regions),
                    "loop": "two buffer sets, copies on their own streams overlap the neighbouring steps' layer calls"},
            "gpu_launches": B.forward_launch_count(cfg_T, T) * args.steps * len(regions),
            "roofline": roofline, "cpu_baseline": cpu}
    if others is not None:
        line["other_workloads"] = others
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# launch path
# ------------------------------------------------------------------------------------------------
def _free_port():
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def replica_command(n, argv, port=None):
    """The command that starts n replica processes of this script on one node (one rank per GPU)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port or _free_port()),
            os.path.abspath(__file__), *argv]


def run_selfcheck(args):
    """Launch-path check without a GPU: every rank joins a gloo group, reports a made-up step time that grows
    with its rank, and rank 0 prints the job line the real arm would print for those times."""
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = max_over_ranks(1.0 + rank, dist if world > 1 else None, torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"impl": "selfcheck", "n_gpus": world, "ms_per_step": ms,
                          "value": job_tokens_per_s(64, world, ms), "unit": UNIT}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "selfcheck"])
    ap.add_argument("--workload", default="mixtral_decode", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--tokens", type=int, default=0,
                    help="tokens per step (default: the largest batch size of the workload, 64 for mixtral_decode)")
    ap.add_argument("--path", default="auto", choices=["auto", "cuda_core", "tensor"])
    ap.add_argument("--layers", type=int, default=0,
                    help="mixtral_stack only: layers per step (default: the workload's 32; 46 GB of packed experts)")
    ap.add_argument("--no-graph", action="store_true", help="mixtral_stack only: launch eagerly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--scale-mode", type=int, default=0, choices=[0, 1],
                    help="0: tied residual scales; 1: free per-step scales (Eq. 4 / Eq. 5)")
    ap.add_argument("--min-region-s", type=float, default=1.0,
                    help="repeat the timed K-step region until this much device time has been timed")
    ap.add_argument("--others", default="all", choices=["all", "layers", "none"],
                    help="after the headline, short legs of the other configurations (default workload, one GPU): "
                         "all = single-layer ones and the 32-layer stack, layers = single-layer ones only")
    args = ap.parse_args()
    if args.others == "none":
        args.others = ""
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    world = int(os.environ.get("WORLD_SIZE", "0"))
    if args.gpus > 1 and world == 0 and args.impl != "reference":
        # started as a plain script: start the replicas ourselves (one process per GPU) and pass their line on
        import subprocess
        sys.exit(subprocess.run(replica_command(args.gpus, sys.argv[1:])).returncode)
    if args.impl == "reference":
        run_reference(args)
    elif args.impl == "selfcheck":
        run_selfcheck(args)
    elif synth.WORKLOADS[args.workload].n_layers > 1 and world <= 1:
        run_stack(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
