"""Shared test plumbing: the same seeded layer, once as packed device blobs for the CUDA path and once
as oracle MWQ tensors on the CPU.  No method arithmetic lives here: every quantization, dequantization,
FFN and combine below is a call into ``oracle/``; this file only cuts the work into pieces (which
tokens, which expert on which thread) and adds the pieces the oracle returned."""
from __future__ import annotations

import os
import threading
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Iterable, List, Optional, Sequence, Tuple

import numpy as np
import torch

from paper_2504_15299_b200 import synth


def np_f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy()


def gpu_layer(binding, cfg, wl, layer: int = 0, device="cuda"):
    """Packed blobs [expert][gate, up, down] generated and packed on the device, one matrix at a time."""
    blobs = []
    for e in range(wl.n_experts + wl.n_shared):
        for m in range(3):
            W = synth.expert_matrix(wl, e, m, device=device, layer=layer)
            blobs.append(binding.pack_mwq(cfg, W))
            del W
    torch.cuda.synchronize()
    return blobs


class OracleLayer:
    """Oracle-side experts, quantized lazily from the same seeded weights (CPU)."""

    def __init__(self, wl, layer: int = 0, scale_mode: int = 0):
        from oracle import mwq
        self.wl, self.layer, self._mwq, self.scale_mode = wl, layer, mwq, scale_mode
        self.cache = {}
        self.raw_cache = {}

    def raw(self, e: int):
        if e not in self.raw_cache:
            self.raw_cache[e] = tuple(np_f32(synth.expert_matrix(self.wl, e, m, layer=self.layer)) for m in range(3))
        return self.raw_cache[e]

    def __call__(self, e: int):
        if e not in self.cache:
            self.cache[e] = tuple(self._mwq.quantize(W, self.wl.bits, self.wl.group_size, self.scale_mode)
                                  for W in self.raw(e))
            self.raw_cache.pop(e, None)
        return self.cache[e]


def max_norm_rel_err(y_gpu: np.ndarray, y_ref: np.ndarray) -> float:
    """max_i |y_gpu[i] - y_ref[i]| / max_i |y_ref[i]| for one token row."""
    return float(np.max(np.abs(y_gpu.astype(np.float64) - y_ref)) / max(np.max(np.abs(y_ref)), 1e-30))


def elementwise_excess(y_gpu: np.ndarray, y_ref: np.ndarray, rel: float = 1e-2) -> float:
    """Largest |delta_i| / (rel |y_ref_i| + rel rms(y_ref)) over one token row: <= 1 means every element
    is within rel of its own magnitude plus rel of the row's rms (small elements are checked too)."""
    y_ref = np.asarray(y_ref, dtype=np.float64)
    d = np.abs(y_gpu.astype(np.float64) - y_ref)
    rms = float(np.sqrt(np.mean(y_ref * y_ref)))
    return float(np.max(d / (rel * np.abs(y_ref) + rel * rms + 1e-300)))


def check_rows(y_gpu: np.ndarray, ref: Dict[int, np.ndarray], tol: float = 1e-2) -> Tuple[float, float]:
    """Both metrics over the reference rows: (worst max-norm relative error, worst element-wise excess).
    An all-zero reference row must come out as exact zeros."""
    worst_mn = worst_el = 0.0
    for t, row in ref.items():
        if np.abs(row).max() == 0.0:
            assert np.abs(y_gpu[t]).max() == 0.0, t
            continue
        worst_mn = max(worst_mn, max_norm_rel_err(y_gpu[t], row))
        worst_el = max(worst_el, elementwise_excess(y_gpu[t], row, tol))
    return worst_mn, worst_el


# ------------------------------------------------------------------------------------------------
# oracle on a token sample of a full-size layer
# ------------------------------------------------------------------------------------------------
def group_edge_tokens(rt, top_k: int, extra: int = 0) -> List[int]:
    """Deterministic token sample of one routed batch: the tokens of the first and the last member of
    every non-empty (expert, width) group, plus `extra` tokens spread evenly over the batch."""
    gr = rt.grouping
    toks = set()
    for key in range(len(gr.group_off) - 1):
        a0, a1 = int(gr.group_off[key]), int(gr.group_off[key + 1])
        if a1 > a0:
            toks.add(int(gr.perm[a0]) // top_k)
            toks.add(int(gr.perm[a1 - 1]) // top_k)
    T = rt.topk_idx.shape[0]
    for i in range(extra):
        toks.add((i * T) // max(extra, 1))
    return sorted(toks)


def oracle_threads() -> int:
    n = int(os.environ.get("D2MOE_ORACLE_THREADS", "0"))
    return n if n > 0 else max(1, min(16, (os.cpu_count() or 2) - 1))


def oracle_sampled(wl, jobs: Sequence[Tuple[np.ndarray, object, Iterable[int]]], layer: int = 0,
                   gen_device: str = "cpu", n_threads: Optional[int] = None, scale_mode: int = 0) -> List[Dict[int, np.ndarray]]:
    """Oracle layer outputs for token samples of several batches that share one layer's weights.

    jobs: (x fp32 [T, d] bf16-exact, oracle Routing of that batch, tokens wanted).  Returns one
    {token: fp64 [d]} per job.

    The layer output is a sum over a token's experts, so the work is cut by expert: for expert e the
    sampled tokens of all jobs that selected e form a one-expert sub-problem (top-1, the token's gate
    weight and routed width), which ``oracle.moe.moe_layer`` computes as it stands; this helper adds
    the per-expert rows in slot order.  Experts run on a thread pool (numpy releases the interpreter
    lock inside its loops), each quantizing its three matrices once.  ``test_oracle_sampled_helper``
    pins the cutting against a direct ``moe_layer`` call on the whole batch.
    """
    from oracle import moe, mwq, routing
    K, k, E = len(wl.bits), wl.top_k, wl.n_experts
    jobs = [(np.ascontiguousarray(x, dtype=np.float32), rt, sorted(set(int(t) for t in toks))) for x, rt, toks in jobs]
    # rows of expert e: (job, token, slot)
    rows_of: Dict[int, List[Tuple[int, int, int]]] = {}
    for j, (x, rt, toks) in enumerate(jobs):
        for t in toks:
            for s in range(k):
                rows_of.setdefault(int(rt.topk_idx[t, s]), []).append((j, t, s))
            for sh in range(wl.n_shared):
                rows_of.setdefault(E + sh, []).append((j, t, -1))
    part: Dict[Tuple[int, int, int], np.ndarray] = {}       # (job, token, slot or -1-shared) -> weighted expert output

    def expert_task(e: int, raw):
        triple = tuple(mwq.quantize(W, wl.bits, wl.group_size, scale_mode) for W in raw)
        del raw
        rows = rows_of[e]
        xs = np.stack([jobs[j][0][t] for j, t, _ in rows])
        n = len(rows)
        if e < E:
            idx = np.zeros((n, 1), dtype=np.int32)
            w = np.array([[jobs[j][1].topk_w[t, s]] for j, t, s in rows], dtype=np.float64)
            bit = np.array([[jobs[j][1].bit_idx[t, s]] for j, t, s in rows], dtype=np.int8)
            sub = routing.Routing(None, idx, w, bit, routing.group_assignments(idx, bit, 1, K))
            out = moe.moe_layer(xs, sub, lambda _e: triple, wl.bits, 1, 0)
        else:
            idx = np.zeros((n, 1), dtype=np.int32)
            sub = routing.Routing(None, idx, np.zeros((n, 1)), np.zeros((n, 1), dtype=np.int8),
                                  routing.group_assignments(np.zeros((0, 1), dtype=np.int32),
                                                            np.zeros((0, 1), dtype=np.int8), 1, K))
            out = moe.moe_layer(xs, sub, lambda _e: triple, wl.bits, 0, 1)
        return {(j, t, s if e < E else -1 - (e - E)): out[i] for i, (j, t, s) in enumerate(rows)}

    n_threads = n_threads or oracle_threads()
    gate = threading.Semaphore(n_threads + 1)                # bounds the raw matrices waiting in memory

    def guarded(e, raw):
        try:
            return expert_task(e, raw)
        finally:
            gate.release()

    # heaviest experts first (more widths to dequantize)
    order = sorted(rows_of, key=lambda e: -len({(jobs[j][1].bit_idx[t, s] if s >= 0 else K) for j, t, s in rows_of[e]}))
    with ThreadPoolExecutor(max_workers=n_threads) as pool:
        futs = []
        for e in order:
            gate.acquire()
            raw = tuple(np_f32(synth.expert_matrix(wl, e, m, device=gen_device, layer=layer)) for m in range(3))
            futs.append(pool.submit(guarded, e, raw))
            del raw
        for f in futs:
            part.update(f.result())

    out: List[Dict[int, np.ndarray]] = []
    for j, (x, rt, toks) in enumerate(jobs):
        res = {}
        for t in toks:
            y = np.zeros(x.shape[1], dtype=np.float64)
            for s in range(k):
                y = y + part[(j, t, s)]
            for sh in range(wl.n_shared):
                y = y + part[(j, t, -1 - sh)]
            res[t] = y
        out.append(res)
    return out
