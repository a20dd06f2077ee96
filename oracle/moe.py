"""Oracle: expert FFN at the routed width, weighted combine, layer stack.  Test infrastructure only.

For every (token, selected expert) pair the expert runs on its weights dequantized at the width
the bit-width router chose (Fig. 1: each token gets an expert id and a bit-width; Section 3.3.1:
"tensors are dequantized ... to enable matrix multiplication with activations").  The experts are
the SwiGLU feed-forward blocks of the evaluated models (Section 5.1), no bias; the layer output is
the gate-weighted sum over the selected experts.  Shared experts (not in the paper; one benchmark
configuration has them) are always on, run at the top width and are added with weight 1.

Everything here is fp64 on exactly-dequantized weights and bf16-exact inputs, with no rounding of
the intermediate activation h.
"""
from __future__ import annotations

from typing import Callable, Dict, Iterable, Optional, Sequence, Tuple

import numpy as np

from . import mwq
from .routing import Routing

ExpertTriple = Tuple[mwq.MWQTensor, mwq.MWQTensor, mwq.MWQTensor]   # gate [F,d], up [F,d], down [d,F]


def swiglu_ffn(x: np.ndarray, Wg: np.ndarray, Wu: np.ndarray, Wd: np.ndarray) -> np.ndarray:
    """o = Wd ( silu(Wg x) * (Wu x) ) for each row x of ``x`` (fp64)."""
    g = x @ Wg.T
    u = x @ Wu.T
    h = g / (1.0 + np.exp(-g)) * u
    return h @ Wd.T


def expert_at_width(x: np.ndarray, expert: ExpertTriple, b: int) -> np.ndarray:
    """Expert output for token rows x with all three matrices dequantized at width b."""
    qg, qu, qd = expert
    x = np.asarray(x, dtype=np.float64)
    g = x @ mwq.dequantize(qg, b).T
    u = x @ mwq.dequantize(qu, b).T
    h = g / (1.0 + np.exp(-g)) * u
    return h @ mwq.dequantize(qd, b).T


def moe_layer(x: np.ndarray, routing: Routing, get_expert: Callable[[int], ExpertTriple],
              bits: Sequence[int], n_experts: int, n_shared: int = 0,
              tokens: Optional[Iterable[int]] = None) -> Dict[int, np.ndarray]:
    """Layer output y_t = sum_slot w[t,slot] * Expert_{e, b}(x_t) (+ shared experts) in fp64.

    Walks the (expert, width) groups of ``routing.grouping`` so each expert is dequantized once per
    width in use.  ``tokens`` limits the computation to a subset of token rows (all by default).
    Returns {token index: fp64 [d] output row}.
    """
    x = np.asarray(x, dtype=np.float64)
    T, d = x.shape
    k = routing.topk_idx.shape[1]
    K = len(bits)
    want = set(range(T)) if tokens is None else set(int(t) for t in tokens)
    y = {t: np.zeros(d, dtype=np.float64) for t in want}
    gr = routing.grouping
    for e in range(n_experts):
        expert = None
        for kk in range(K):
            key = e * K + kk
            members = [int(a) for a in gr.perm[gr.group_off[key]:gr.group_off[key + 1]] if int(a) // k in want]
            if not members:
                continue
            if expert is None:
                expert = get_expert(e)
            ts = [a // k for a in members]
            o = expert_at_width(x[ts], expert, bits[kk])
            for row, a in enumerate(members):
                t, slot = divmod(a, k)
                assert routing.topk_idx[t, slot] == e and routing.bit_idx[t, slot] == kk
                y[t] += routing.topk_w[t, slot] * o[row]
    for s in range(n_shared):
        expert = get_expert(n_experts + s)
        ts = sorted(want)
        if ts:
            o = expert_at_width(x[ts], expert, bits[-1])
            for row, t in enumerate(ts):
                y[t] += o[row]
    return y


def round_to_bf16(v: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to bf16, returned as fp32 values."""
    f = np.ascontiguousarray(v, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    rounded = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return rounded.astype(np.uint32).view(np.float32).reshape(f.shape)


def rmsnorm(x: np.ndarray, eps: float = 1e-5) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) per row (unit gain), fp64."""
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt((x * x).mean(axis=1, keepdims=True) + eps)


def stack_layer(x: np.ndarray, moe_of_normed: Callable[[np.ndarray], np.ndarray]) -> np.ndarray:
    """One layer of the FFN-only stack: x <- bf16( x + MoE( bf16( RMSNorm(x) ) ) )."""
    xn = round_to_bf16(rmsnorm(x)).astype(np.float64)
    return round_to_bf16(np.asarray(x, dtype=np.float64) + moe_of_normed(xn)).astype(np.float64)


def unquantized_moe_layer(x: np.ndarray, routing: Routing,
                          get_weights: Callable[[int], Tuple[np.ndarray, np.ndarray, np.ndarray]],
                          n_experts: int, n_shared: int = 0) -> np.ndarray:
    """Brute-force MoE on the original fp32 weights (no quantization), token by token, fp64.
    Only used to check that the 8-bit layer stays within the INT8 error bound."""
    x = np.asarray(x, dtype=np.float64)
    T, d = x.shape
    k = routing.topk_idx.shape[1]
    y = np.zeros((T, d), dtype=np.float64)
    cache = {}
    for t in range(T):
        experts = [(int(routing.topk_idx[t, s]), float(routing.topk_w[t, s])) for s in range(k)]
        experts += [(n_experts + s, 1.0) for s in range(n_shared)]
        for e, w in experts:
            if e not in cache:
                cache[e] = tuple(np.asarray(m, dtype=np.float64) for m in get_weights(e))
            Wg, Wu, Wd = cache[e]
            y[t] += w * swiglu_ffn(x[t:t + 1], Wg, Wu, Wd)[0]
    return y
