#!/usr/bin/env python
"""Benchmark of the dual-routed MWQ MoE layer (one step = one pass of the whole hot path over one batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload mixtral_decode] [--tokens 64] [--path auto|cuda_core|tensor]

Prints ONE JSON line.  N > 1 runs independent replicas, one process per GPU (launched by
torch.distributed.run), no data-path collective; the barrier and the max-over-ranks timing use NCCL.
`--impl reference` times the CPU oracle on the host cores on a bounded sample of the same workload.
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
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from one ncu capture of
# this command (profiles/ffn_i8_kernel_mixtral_decode_T64.md); key = workload:tokens:stage:path
NCU_TRAFFIC = {"mixtral_decode:T64:gate_up:auto": 1044382432, "mixtral_decode:T64:down:auto": 539915144}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def measured_tensor_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["bf16_tflops_sustained"]), "measured (sustained)"
        except Exception:
            pass
    return 1400.0, "fallback (sustained)"


# ------------------------------------------------------------------------------------------------
# algorithmic bytes: what the method has to read at the routed widths - per active expert and matrix the
# packed prefix up to the widest width routed to that expert in this call, read once, plus activations
# in and outputs out
# ------------------------------------------------------------------------------------------------
def matrix_bytes(rows, cols, g, bits_read):
    return rows * cols * bits_read // 8 + rows * (cols // g) * 4


def algorithmic_bytes(wl, T, group_off):
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
        gu += 2 * matrix_bytes(wl.d_ffn, wl.d_model, wl.group_size, b)
        dn += matrix_bytes(wl.d_model, wl.d_ffn, wl.group_size, b)
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


def workload_config(wl, T, path):
    return {"workload": f"{wl.name} T={T}: d={wl.d_model} ffn={wl.d_ffn} E={wl.n_experts} top{wl.top_k} "
                        f"g={wl.group_size} bits={list(wl.bits)} p={list(wl.bit_probs)}",
            "tokens_per_step": T, "kernel_path": path,
            "l2": "inputs larger than L2: each step streams the routed planes of every active expert "
                  "(>1 GB per layer call against a 126 MB L2); four token batches are rotated"}


# ------------------------------------------------------------------------------------------------
# layer stack (the 32-layer decode configuration): one step = every layer once, replayed as a CUDA graph
# ------------------------------------------------------------------------------------------------
def run_stack(args):
    from paper_2504_15299_b200 import binding as B, build
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    build.build_library()
    B.lib()
    wl = synth.WORKLOADS[args.workload]
    T = args.tokens or wl.tokens[-1]
    L = args.layers or wl.n_layers
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
    if not args.no_graph:
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

    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms_per_step = e0.elapsed_time(e1) / args.steps
    assert int(status.item()) == 0, f"device status {int(status.item())}"

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
    for i in range(args.steps):
        e2e_step(i)
    f1.record()
    torch.cuda.synchronize()
    e2e_ms = f0.elapsed_time(f1) / args.steps

    peak, peak_kind = measured_peaks()
    achieved = step_bytes / (ms_per_step * 1e-3) / 1e9
    line = {"metric": METRIC, "value": T / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "i8", "data": "synthetic",
            "config": {"workload": f"{wl.name}: {L} layers of d={wl.d_model} ffn={wl.d_ffn} E={wl.n_experts} "
                                   f"top{wl.top_k} g={wl.group_size} bits={list(wl.bits)}, widths from the per-expert "
                                   f"bit-width routers, RMSNorm + residual per layer",
                       "tokens_per_step": T, "layers": L, "cuda_graph": graph is not None,
                       "l2": f"inputs larger than L2: {L} layers of distinct packed experts "
                             f"({step_bytes / 1e9:.1f} GB read per step)"},
            "clocks": clocks,
            "e2e": {"value": T / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": hx[0].numel() * 2,
                    "d2h_bytes_per_step": hy.numel() * 2},
            "gpu_launches": (B.forward_launch_count(cfg, T) + 1) * L * args.steps,
            "roofline": {"bound": "hbm", "kernel": "whole step", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": None,
                         "algorithmic_bytes_per_step": step_bytes},
            "cpu_baseline": None}
    print(json.dumps(line))


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
    path = {"auto": B.PATH_AUTO, "cuda_core": B.PATH_CUDA_CORE, "tensor": B.PATH_TENSOR}[args.path]
    cfg = B.Config.from_workload(wl, kernel_path=path)

    blobs = []
    for e in range(wl.n_experts + wl.n_shared):
        for m in range(3):
            W = synth.expert_matrix(wl, e, m, device=dev)
            blobs.append(B.pack_mwq(cfg, W))
            del W
    gw = synth.gate_weight_bf16(wl, dev)
    n_batches = 4
    xs = [synth.tokens_bf16(wl, T, dev, step=rank * 100 + i) for i in range(n_batches)]
    fbs = [synth.categorical(wl.seed + rank * 100 + i, synth.TID_FORCED_BITS, (T, wl.top_k), wl.bit_probs, dev)
           for i in range(n_batches)]
    logits = [synth.zipf_logits(wl, T, dev) for _ in range(n_batches)] if wl.zipf_logits else None
    ws = torch.empty(B.workspace_bytes(cfg, T), dtype=torch.uint8, device=dev)
    y = torch.empty_like(xs[0])
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def kw(i):
        d = {"forced_bit_idx": fbs[i]}
        if logits is not None:
            d["logits"] = logits[i]
        else:
            d["gate_w"] = gw
        return d

    # realised routing of each batch -> algorithmic bytes
    alg = []
    for i in range(n_batches):
        r = B.route(cfg, xs[i], workspace=ws, **kw(i))
        torch.cuda.synchronize()
        alg.append(algorithmic_bytes(wl, T, r.group_off.cpu().tolist()))

    def step(i, events=None):
        B.moe_forward(cfg, xs[i % n_batches], blobs, y=y, workspace=ws, device_status=status,
                      stage_events=events, **kw(i % n_batches))

    def sync_all():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    sync_all()

    # ---- timed region: K steps, device time, max over ranks ----
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    stream = torch.cuda.current_stream()
    stage_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(B.N_STAGES + 1)] for _ in range(args.steps)]
    for evs in stage_ev:
        for ev in evs:
            ev.record(stream)            # creates the handle
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    # per-stage events on every fifth step (with four batches in rotation every batch gets its share):
    # recording five events per step costs about 3 % of a decode step, and the stage times are averages
    # over the timed region anyway
    ev_steps = [i for i in range(args.steps) if i % 5 == 0 or args.steps < 10]
    for i in range(args.steps):
        step(i, stage_ev[i] if (i % 5 == 0 or args.steps < 10) else None)
    e1.record(stream)
    sync_all()
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step = max_over_ranks(e0.elapsed_time(e1), dist, dev) / args.steps
    assert int(status.item()) == 0, f"device status {int(status.item())}"

    stage_ms = [sum(stage_ev[i][s].elapsed_time(stage_ev[i][s + 1]) for i in ev_steps) / len(ev_steps)
                for s in range(B.N_STAGES)]

    # ---- end to end: pinned host inputs -> device, layer, result back to the host, every step ----
    # The serving loop a user of the library would write: two sets of device buffers, the copies on streams of
    # their own, so that the copy-in of step i + 1 and the copy-out of step i - 1 overlap the layer call of
    # step i.  Every step's inputs come from pinned host memory and every step's result lands in pinned host
    # memory inside the timed region; the region ends when the last result has arrived.
    hx = [x.cpu().pin_memory() for x in xs]
    hfb = [f.cpu().pin_memory() for f in fbs]
    hy = [torch.empty_like(hx[0]).pin_memory() for _ in range(2)]
    dx = [torch.empty_like(xs[0]) for _ in range(2)]
    dfb = [torch.empty_like(fbs[0]) for _ in range(2)]
    dy = [torch.empty_like(y) for _ in range(2)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]       # inputs of the buffer set have arrived
    ev_done = [torch.cuda.Event() for _ in range(2)]     # the layer call on the buffer set has finished
    ev_out = [torch.cuda.Event() for _ in range(2)]      # its result has left the device
    for b in range(2):
        ev_done[b].record(stream)
        ev_out[b].record(stream)

    def e2e_step(i):
        j, b = i % n_batches, i & 1
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_done[b])                   # the call two steps back has read these inputs
            dx[b].copy_(hx[j], non_blocking=True)
            dfb[b].copy_(hfb[j], non_blocking=True)
            ev_in[b].record(s_in)
        stream.wait_event(ev_in[b])
        stream.wait_event(ev_out[b])                      # the result two steps back has been copied out
        d = {"forced_bit_idx": dfb[b]}
        if logits is not None:
            d["logits"] = logits[j]
        else:
            d["gate_w"] = gw
        B.moe_forward(cfg, dx[b], blobs, y=dy[b], workspace=ws, device_status=status, **d)
        ev_done[b].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[b])
            hy[b].copy_(dy[b], non_blocking=True)
            ev_out[b].record(s_out)

    for i in range(args.warmup):
        e2e_step(i)
    sync_all()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for i in range(args.steps):
        e2e_step(args.warmup + i)
    stream.wait_event(ev_out[0])
    stream.wait_event(ev_out[1])
    f1.record(stream)
    sync_all()
    e2e_ms = max_over_ranks(f0.elapsed_time(f1), dist, dev) / args.steps

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    used = [alg[i % n_batches] for i in ev_steps]          # the steps whose stages were timed
    stage_names = B.STAGE_NAMES
    dom = max(range(B.N_STAGES), key=lambda s: stage_ms[s])
    dom_name = stage_names[dom]
    dom_bytes = sum(u.get(dom_name, u["layer"]) for u in used) / len(used)
    layer_bytes = sum(u["layer"] for u in used) / len(used)
    achieved = dom_bytes / (stage_ms[dom] * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dom_name, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": None,
                "algorithmic_bytes_per_launch": dom_bytes,
                "stage_ms": dict(zip(stage_names, stage_ms)),
                "stage_samples": len(ev_steps),
                "layer": {"algorithmic_bytes": layer_bytes,
                          "achieved_gbs": layer_bytes / (ms_per_step * 1e-3) / 1e9,
                          "frac": layer_bytes / (ms_per_step * 1e-3) / 1e9 / peak}}
    roofline["traffic"] = NCU_TRAFFIC.get(f"{args.workload}:T{T}:{dom_name}:{args.path}")
    # prefill-sized expert loads (the grouped dequant-GEMM) are bound by the tensor cores: report
    # the dominant kernel against the measured dense 16-bit matmul rate instead (fp16 operands have the
    # same nominal rate as the bf16 the peak was measured with; sustained figure: kernel inside a step)
    # arithmetic type of the expert kernels: the decode kernel multiplies unsigned 8-bit codes with signed
    # 8-bit activation halves (int32 accumulation, fp32 scaling), the grouped GEMM runs on fp16 tiles
    dtype = "f32" if args.path == "cuda_core" else "i8"
    if -(-T * wl.top_k // wl.n_experts) > 40 and args.path != "cuda_core":
        dtype = "f16"
        A_tot = T * (wl.top_k + wl.n_shared)
        flops = {"gate_up": A_tot * 2 * 2 * wl.d_model * wl.d_ffn, "down": A_tot * 2 * wl.d_model * wl.d_ffn}
        tpeak, tkind = measured_tensor_peak()
        tf = flops.get(dom_name, sum(flops.values())) / (stage_ms[dom] * 1e-3) / 1e12
        roofline.update({"bound": "tensor", "achieved": tf, "peak": tpeak, "unit": "TFLOP/s",
                         "frac": tf / tpeak, "peak_kind": f"of {tkind}", "traffic": None,
                         "algorithmic_flops_per_launch": flops.get(dom_name)})
        roofline["layer"] = {"algorithmic_flops": sum(flops.values()),
                             "achieved_tflops": sum(flops.values()) / (ms_per_step * 1e-3) / 1e12,
                             "frac": sum(flops.values()) / (ms_per_step * 1e-3) / 1e12 / tpeak}

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        v, per, hid = oracle_tokens_per_s(wl, T, 1, 32, 2, 0, device_for_inputs=dev)
        cpu = {"value": v, "unit": UNIT, "cores": used_threads(), "kind": "oracle",
               "sample": f"first token of the batch, all its experts at the routed widths, hidden units "
                         f"0..{hid - 1} of {wl.d_ffn} per expert, time scaled by {wl.d_ffn}/{hid} "
                         f"(extrapolated); 2 passes"}

    line = {"metric": METRIC, "value": job_tokens_per_s(T, world, ms_per_step), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": dtype,
            "data": "synthetic", "config": workload_config(wl, T, args.path),
            "clocks": clocks,
            "e2e": {"value": job_tokens_per_s(T, world, e2e_ms), "unit": UNIT,
                    "h2d_bytes_per_step": hx[0].numel() * 2 + hfb[0].numel(),
                    "d2h_bytes_per_step": hy[0].numel() * 2,
                    "loop": "two buffer sets, copies on their own streams overlap the neighbouring steps' layer calls; "
                            "no per-stage events in this loop (the device-timed loop records five per step)"},
            "gpu_launches": B.forward_launch_count(cfg, T) * args.steps,
            "roofline": roofline, "cpu_baseline": cpu}
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mixtral_decode", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--tokens", type=int, default=0,
                    help="tokens per step (default: the largest batch size of the workload, 64 for mixtral_decode)")
    ap.add_argument("--path", default="auto", choices=["auto", "cuda_core", "tensor"])
    ap.add_argument("--layers", type=int, default=0,
                    help="mixtral_stack only: layers per step (default: the workload's 32; 46 GB of packed experts)")
    ap.add_argument("--no-graph", action="store_true", help="mixtral_stack only: launch eagerly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif synth.WORKLOADS[args.workload].n_layers > 1 and int(os.environ.get("WORLD_SIZE", "1")) == 1:
        run_stack(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
