"""Shared test plumbing: the same seeded layer, once as packed device blobs for the CUDA path and once
as oracle MWQ tensors on the CPU.  No method arithmetic lives here."""
from __future__ import annotations

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

    def __init__(self, wl, layer: int = 0):
        from oracle import mwq
        self.wl, self.layer, self._mwq = wl, layer, mwq
        self.cache = {}
        self.raw_cache = {}

    def raw(self, e: int):
        if e not in self.raw_cache:
            self.raw_cache[e] = tuple(np_f32(synth.expert_matrix(self.wl, e, m, layer=self.layer)) for m in range(3))
        return self.raw_cache[e]

    def __call__(self, e: int):
        if e not in self.cache:
            self.cache[e] = tuple(self._mwq.quantize(W, self.wl.bits, self.wl.group_size) for W in self.raw(e))
            self.raw_cache.pop(e, None)
        return self.cache[e]


def max_norm_rel_err(y_gpu: np.ndarray, y_ref: np.ndarray) -> float:
    """max_i |y_gpu[i] - y_ref[i]| / max_i |y_ref[i]| for one token row."""
    return float(np.max(np.abs(y_gpu.astype(np.float64) - y_ref)) / max(np.max(np.abs(y_ref)), 1e-30))
