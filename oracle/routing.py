"""Oracle: dual routing (Section 3.2; models of Section 5.1) and grouping.  Test infrastructure only.

Each token goes through the expert gate (top-k of E experts) and, for every selected expert,
through that expert's bit-width router, which picks one of the K candidate widths
(Section 3.2, "a lightweight, trainable bit-width router is placed before each expert").
The per-layer count of selections per (expert, width) is the matrix B_{j,k} of Section 3.4.3;
sorting the (token, expert) assignments by (expert, width) is the grouping the expert kernels use.

Readings where the paper is silent:
* Gate: top-k on the raw logits (ties go to the lower expert index), softmax over all E logits,
  weights of the selected experts divided by their sum when ``renormalize`` is set (the
  Mixtral / LLaMA-MoE convention of the models the paper evaluates).
* Bit-width router: one bias-free linear map d -> K per expert applied to the expert's input token;
  the width is the argmax of its logits (ties go to the lower width); the expert output is not
  scaled by the router's probability; no capacity dropping at inference (the capacity c_k is a
  fine-tuning device).  PARITY UNPINNED: the paper states neither the router's architecture nor
  its sizes.
* Logits are fp32 in a pinned summation order so that near-ties resolve identically everywhere:
  32 partial sums, partial l takes elements l, l+32, ... in ascending order with one fused
  multiply-add each, then a butterfly reduction (offsets 16, 8, 4, 2, 1).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np

F32 = np.float32


def _is_bf16_exact(a: np.ndarray) -> bool:
    return bool(np.all((np.ascontiguousarray(a, dtype=F32).view(np.uint32) & 0xFFFF) == 0))


def logits_pinned(x: np.ndarray, W: np.ndarray) -> np.ndarray:
    """l[t, e] = sum_i x[t, i] * W[e, i] in fp32, pinned order.  x, W hold bf16-exact values, so
    every product is exact in fp32 and a fused multiply-add equals an fp32 add of the product."""
    x = np.ascontiguousarray(x, dtype=F32)
    W = np.ascontiguousarray(W, dtype=F32)
    assert _is_bf16_exact(x) and _is_bf16_exact(W)
    T, d = x.shape
    E = W.shape[0]
    out = np.empty((T, E), dtype=F32)
    n_steps = (d + 31) // 32
    for e in range(E):
        prod = (x * W[e][None, :]).astype(F32)                    # exact
        if d % 32:
            prod = np.concatenate([prod, np.zeros((T, 32 - d % 32), dtype=F32)], axis=1)
        prod = prod.reshape(T, n_steps, 32)
        acc = np.zeros((T, 32), dtype=F32)
        for m in range(n_steps):
            acc = (acc + prod[:, m, :]).astype(F32)
        lanes = np.arange(32)
        for off in (16, 8, 4, 2, 1):
            acc = (acc + acc[:, lanes ^ off]).astype(F32)
        out[:, e] = acc[:, 0]
    return out


def topk_select(logits: np.ndarray, k: int) -> np.ndarray:
    """k rounds of "take the largest remaining logit", ties to the lower index. int32 [T, k]."""
    T, E = logits.shape
    assert 1 <= k <= E
    idx = np.empty((T, k), dtype=np.int32)
    for t in range(T):
        taken = [False] * E
        for s in range(k):
            best = -1
            for e in range(E):
                if taken[e]:
                    continue
                if best < 0 or logits[t, e] > logits[t, best]:
                    best = e
            taken[best] = True
            idx[t, s] = best
    return idx


def gate_weights(logits: np.ndarray, idx: np.ndarray, renormalize: bool) -> np.ndarray:
    """Softmax over all experts (fp64), gathered at the selected experts. fp64 [T, k]."""
    l = logits.astype(np.float64)
    p = np.exp(l - l.max(axis=1, keepdims=True))
    p = p / p.sum(axis=1, keepdims=True)
    w = np.take_along_axis(p, idx.astype(np.int64), axis=1)
    if renormalize:
        w = w / w.sum(axis=1, keepdims=True)
    return w


def bit_width_choice(x: np.ndarray, Wb: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """Width index per (token, selected expert): argmax of the expert's bit-width router logits
    u[kk] = Wb[e, kk, :] . x_t (pinned fp32 order), first maximum wins.  int8 [T, k].
    PARITY UNPINNED (see module docstring)."""
    T, k = idx.shape
    E, K, d = Wb.shape
    u_all = logits_pinned(x, Wb.reshape(E * K, d)).reshape(T, E, K)
    out = np.empty((T, k), dtype=np.int8)
    for t in range(T):
        for s in range(k):
            u = u_all[t, idx[t, s]]
            best = 0
            for kk in range(1, K):
                if u[kk] > u[best]:
                    best = kk
            out[t, s] = best
    return out


@dataclass
class Grouping:
    hist: np.ndarray       # int32 [E, K]   B_{j,k}: selections per (expert, width)
    group_off: np.ndarray  # int32 [E*K+1]  exclusive prefix sum of hist (row-major)
    perm: np.ndarray       # int32 [A]      sorted position -> flat assignment id a = t*k + slot
    inv_perm: np.ndarray   # int32 [A]      flat assignment id -> sorted position


def group_assignments(idx: np.ndarray, bit_idx: np.ndarray, E: int, K: int) -> Grouping:
    """Stable counting sort of the assignments by key (expert, width index)."""
    T, k = idx.shape
    A = T * k
    hist = np.zeros((E, K), dtype=np.int32)
    for t in range(T):
        for s in range(k):
            hist[idx[t, s], bit_idx[t, s]] += 1
    group_off = np.zeros(E * K + 1, dtype=np.int32)
    for key in range(E * K):
        group_off[key + 1] = group_off[key] + hist[key // K, key % K]
    cursor = group_off[:-1].copy()
    perm = np.empty(A, dtype=np.int32)
    inv_perm = np.empty(A, dtype=np.int32)
    for a in range(A):
        t, s = divmod(a, k)
        key = int(idx[t, s]) * K + int(bit_idx[t, s])
        pos = cursor[key]
        cursor[key] += 1
        perm[pos] = a
        inv_perm[a] = pos
    return Grouping(hist, group_off, perm, inv_perm)


@dataclass
class Routing:
    logits: np.ndarray     # fp32 [T, E]
    topk_idx: np.ndarray   # int32 [T, k]
    topk_w: np.ndarray     # fp64 [T, k]
    bit_idx: np.ndarray    # int8 [T, k]
    grouping: Grouping


def route(x: np.ndarray, *, E: int, K: int, top_k: int, renormalize: bool,
          gate_w: Optional[np.ndarray] = None, logits: Optional[np.ndarray] = None,
          bit_w: Optional[np.ndarray] = None, forced_bit_idx: Optional[np.ndarray] = None) -> Routing:
    """Dual routing of a token batch.  Exactly one of (gate_w, logits) and one of
    (bit_w, forced_bit_idx) is given."""
    assert (gate_w is None) != (logits is None)
    assert (bit_w is None) != (forced_bit_idx is None)
    if logits is None:
        logits = logits_pinned(x, gate_w)
    logits = np.asarray(logits, dtype=F32)
    idx = topk_select(logits, top_k)
    w = gate_weights(logits, idx, renormalize)
    if forced_bit_idx is not None:
        bit_idx = np.asarray(forced_bit_idx, dtype=np.int8).reshape(idx.shape)
    else:
        bit_idx = bit_width_choice(x, bit_w, idx)
    return Routing(logits, idx, w, bit_idx, group_assignments(idx, bit_idx, E, K))
