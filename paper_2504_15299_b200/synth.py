"""Seeded synthetic inputs for the dual-routed MWQ MoE layer.

This module only makes *data*: it holds none of the method's arithmetic (no quantizer, no
router, no FFN).  Both the CPU oracle's tests and the CUDA path draw their inputs from here, so
the two sides see bit-identical tensors.

Every value is a pure function of ``(seed, tensor_id, flat element index)`` through a
counter-based 64-bit integer mixer, so any slice of any tensor (for instance a few sampled
rows of a 58.7 M-element expert matrix) can be regenerated on its own, on the CPU or on the
GPU, without generating the rest.  All steps up to the last are integer operations; the last
steps are a table lookup and three IEEE fp32 operations (sub, mul, add) plus one fp32 multiply
by sigma, each a separate un-fused elementwise op, so CPU and CUDA results are identical.

"N(0, sigma)" here means: inverse-CDF sampling on a 2^16-cell grid of the standard normal
(cell edges are exact quantiles, tails clipped at +-4.5), with linear interpolation inside a
cell driven by 16 further random bits, times sigma.

The workload recipes below restate the five benchmark configurations (shapes, widths, bit
probabilities, seeds).  They stand in for the paper's Mixtral-8x7B / LLaMA-MoE workloads
(Section 5.1: 8 experts, top-2, group size 128): same layer shapes, random-init weights.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from functools import lru_cache
from typing import Optional, Sequence, Tuple

import torch

_M64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Python int (mod 2^64) -> the signed value torch.int64 uses for the same bits."""
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_MUL1 = _s64(0xBF58476D1CE4E5B9)
_MUL2 = _s64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor (torch's >> is arithmetic)."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix64_py(z: int) -> int:
    z &= _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def _mix64(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def stream_key(seed: int, tensor_id: int) -> int:
    """Per-tensor 64-bit key (python int)."""
    return _mix64_py(_mix64_py(seed * 0x9E3779B97F4A7C15 + 0x1234567) + tensor_id * 0xD1B54A32D192ED03)


def random_bits(seed: int, tensor_id: int, index: torch.Tensor) -> torch.Tensor:
    """64 random bits (as int64) for every flat element index in ``index`` (int64 tensor)."""
    key = _s64(stream_key(seed, tensor_id))
    return _mix64(index * _GOLDEN + key)


@lru_cache(maxsize=None)
def _normal_edges_cpu() -> torch.Tensor:
    p = torch.arange(1, 65536, dtype=torch.float64) / 65536.0
    inner = torch.special.ndtri(p)
    edges = torch.cat([torch.tensor([-4.5], dtype=torch.float64), inner,
                       torch.tensor([4.5], dtype=torch.float64)])
    return edges.to(torch.float32)


_EDGE_CACHE = {}


def _normal_edges(device) -> torch.Tensor:
    dev = torch.device(device)
    key = str(dev)
    if key not in _EDGE_CACHE:
        _EDGE_CACHE[key] = _normal_edges_cpu().to(dev)
    return _EDGE_CACHE[key]


def _flat_index(shape: Sequence[int], rows, cols, device) -> Tuple[torch.Tensor, Tuple[int, ...]]:
    """Flat indices of the whole tensor, or of the listed rows / columns of a 2-D tensor."""
    if rows is None and cols is None:
        n = 1
        for s in shape:
            n *= int(s)
        return torch.arange(n, dtype=torch.int64, device=device), tuple(int(s) for s in shape)
    assert len(shape) == 2, "row / column sampling is for 2-D tensors"
    n_cols = int(shape[1])
    rows = torch.arange(int(shape[0]), dtype=torch.int64, device=device) if rows is None else \
        torch.as_tensor(rows, dtype=torch.int64, device=device)
    cols = torch.arange(n_cols, dtype=torch.int64, device=device) if cols is None else \
        torch.as_tensor(cols, dtype=torch.int64, device=device)
    idx = rows[:, None] * n_cols + cols[None, :]
    return idx.reshape(-1), (int(rows.numel()), int(cols.numel()))


def normal(seed: int, tensor_id: int, shape: Sequence[int], sigma: float = 1.0,
           device="cpu", rows: Optional[torch.Tensor] = None, cols: Optional[torch.Tensor] = None,
           chunk: int = 1 << 24) -> torch.Tensor:
    """fp32 tensor ~ "N(0, sigma)" as defined in the module docstring; ``rows`` / ``cols`` select a
    sub-matrix of a 2-D tensor (same values as the corresponding entries of the full tensor)."""
    idx_all, out_shape = _flat_index(shape, rows, cols, device)
    edges = _normal_edges(device)
    out = torch.empty(idx_all.numel(), dtype=torch.float32, device=device)
    for s in range(0, idx_all.numel(), chunk):
        idx = idx_all[s:s + chunk]
        h = random_bits(seed, tensor_id, idx)
        cell = _lsr(h, 48)                       # 16 bits
        u = _lsr(h, 32) & 0xFFFF                 # next 16 bits
        frac = (u.to(torch.float32) + 0.5) * (1.0 / 65536.0)   # exact in fp32
        lo = edges[cell]
        width = edges[cell + 1] - lo
        z = lo + frac * width                    # two separate fp32 ops (eager: no fusion)
        out[s:s + chunk] = z * float(sigma)
    return out.reshape(out_shape)


def uniform24(seed: int, tensor_id: int, shape: Sequence[int], device="cpu") -> torch.Tensor:
    idx, out_shape = _flat_index(shape, None, None, device)
    return _lsr(random_bits(seed, tensor_id, idx), 40).reshape(out_shape)


def categorical(seed: int, tensor_id: int, shape: Sequence[int], probs: Sequence[float],
                device="cpu") -> torch.Tensor:
    """int8 tensor of category indices drawn with the given probabilities (integer thresholds)."""
    u = uniform24(seed, tensor_id, shape, device)
    out = torch.zeros(u.shape, dtype=torch.int64, device=device)
    acc = 0.0
    for p in list(probs)[:-1]:
        acc += p
        thr = int(round(acc * (1 << 24)))
        out += (u >= thr).to(torch.int64)
    return out.to(torch.int8)


def bf16_exact(x: torch.Tensor) -> torch.Tensor:
    """Round an fp32 tensor to bf16 (RNE) and return it as bf16."""
    return x.to(torch.bfloat16)


# ----------------------------------------------------------------------------------------------
# Workload recipes
# ----------------------------------------------------------------------------------------------

# tensor ids inside one layer
TID_X = 1
TID_GATE = 2
TID_BITW = 3          # bit-width router weights
TID_FORCED_BITS = 4
TID_LOGITS = 5
TID_EXPERT0 = 100     # expert e, matrix m (0 gate, 1 up, 2 down): TID_EXPERT0 + 3*e + m


@dataclass(frozen=True)
class Workload:
    name: str
    d_model: int
    d_ffn: int
    n_experts: int
    top_k: int
    group_size: int
    bits: Tuple[int, ...]
    bit_probs: Tuple[float, ...]
    seed: int
    n_shared: int = 0
    tokens: Tuple[int, ...] = (16,)
    renormalize: int = 1
    zipf_logits: bool = False      # router logits supplied: N(0,1) + ln(1/(e+1))
    learned_bits: bool = False     # bit-widths come from the per-expert bit-width router
    n_layers: int = 1
    sigma_w: float = 0.02


WORKLOADS = {
    "tiny": Workload("tiny", 256, 512, 4, 2, 64, (2, 4, 8), (1 / 3, 1 / 3, 1 / 3), seed=0, tokens=(16,)),
    "mixtral_decode": Workload("mixtral_decode", 4096, 14336, 8, 2, 128, (2, 3, 4, 8),
                               (0.1, 0.2, 0.4, 0.3), seed=1, tokens=(1, 8, 32, 64)),
    "mixtral_prefill": Workload("mixtral_prefill", 4096, 14336, 8, 2, 128, (2, 3, 4, 8),
                                (0.1, 0.2, 0.4, 0.3), seed=1, tokens=(2048,), zipf_logits=True),
    "finegrained": Workload("finegrained", 2048, 1408, 64, 6, 128, (2, 4, 8), (0.3, 0.4, 0.3),
                            seed=3, n_shared=2, tokens=(256,)),
    "mixtral_stack": Workload("mixtral_stack", 4096, 14336, 8, 2, 128, (2, 3, 4, 8),
                              (0.25, 0.25, 0.25, 0.25), seed=4, tokens=(16,), learned_bits=True,
                              n_layers=32),
    # the same layer shape with the width list {5,6,7,8}, and a dense gated FFN (one expert, top-1) of
    # LLaMA2-13B's FFN shape: both are plain configurations of the same path
    "mixtral_v2": Workload("mixtral_v2", 4096, 14336, 8, 2, 128, (5, 6, 7, 8),
                           (0.25, 0.25, 0.25, 0.25), seed=5, tokens=(64,)),
    "dense_ffn": Workload("dense_ffn", 5120, 13824, 1, 1, 128, (2, 3, 4, 8),
                          (0.1, 0.2, 0.4, 0.3), seed=6, tokens=(16,)),
}


def expert_matrix_shape(wl: Workload, m: int) -> Tuple[int, int]:
    """m = 0 gate projection [F, d], 1 up projection [F, d], 2 down projection [d, F]."""
    return (wl.d_ffn, wl.d_model) if m < 2 else (wl.d_model, wl.d_ffn)


def expert_matrix(wl: Workload, e: int, m: int, device="cpu", layer: int = 0,
                  rows: Optional[torch.Tensor] = None, cols: Optional[torch.Tensor] = None) -> torch.Tensor:
    """fp32 weights ~N(0, sigma_w) of expert ``e`` (shared experts follow the routed ones)."""
    return normal(wl.seed + layer, TID_EXPERT0 + 3 * e + m, expert_matrix_shape(wl, m),
                  wl.sigma_w, device, rows, cols)


def tokens_bf16(wl: Workload, T: int, device="cpu", step: int = 0) -> torch.Tensor:
    seed = wl.seed if step == 0 else 1000 + step
    return bf16_exact(normal(seed, TID_X, (T, wl.d_model), 1.0, device))


def gate_weight_bf16(wl: Workload, device="cpu", layer: int = 0) -> torch.Tensor:
    return bf16_exact(normal(wl.seed + layer, TID_GATE, (wl.n_experts, wl.d_model), wl.sigma_w, device))


def bit_router_weight_bf16(wl: Workload, device="cpu", layer: int = 0) -> torch.Tensor:
    shape = (wl.n_experts * len(wl.bits), wl.d_model)
    w = normal(wl.seed + layer, TID_BITW, shape, wl.sigma_w, device)
    return bf16_exact(w).reshape(wl.n_experts, len(wl.bits), wl.d_model)


def forced_bit_idx(wl: Workload, T: int, device="cpu") -> torch.Tensor:
    return categorical(wl.seed, TID_FORCED_BITS, (T, wl.top_k), wl.bit_probs, device)


def zipf_logits(wl: Workload, T: int, device="cpu") -> torch.Tensor:
    """Router logits N(0,1) + ln(1/(e+1)) (Zipf s=1 prior over experts), fp64 on the host -> fp32."""
    z = normal(wl.seed, TID_LOGITS, (T, wl.n_experts), 1.0, "cpu").to(torch.float64)
    prior = torch.tensor([math.log(1.0 / (e + 1)) for e in range(wl.n_experts)], dtype=torch.float64)
    return (z + prior[None, :]).to(torch.float32).to(device)
