"""Oracle: Matryoshka Weight Quantization (Section 3.3.1).  Test infrastructure only.

Calibration-free form: the paper optimises the zero points and scales against activations X
(Eq. 3, Eq. 5) and compensates block errors through a Hessian factor (Algorithm 1).  No
calibration data exists here; with X proportional to the identity the Hessian factor is diagonal
and the compensation update is zero, so what is left is Eq. 2 followed by the one-bit residual
steps of Eq. 4, which is what this file writes out.

Readings taken where the paper is silent:
* ``round`` in Eq. 2 is round-half-to-even; the base code is clamped to [0, 2^b1 - 1].
* Zero point is real-valued (Eq. 2 has z in R); it is stored as ``lo = -z*s``, an fp16 value rounded
  toward -inf from the group minimum, and the scale ``s1`` is the fp16 value rounded toward +inf
  from (max - lo)/(2^b1 - 1), so the base grid always covers the group.  s1 == 0 becomes 2^-14.
* Eq. 4 with Q in {+1,-1}: Q = sign of the residual, sign(0) = +1.
* Residual scales, default (``scale_mode = 0``): tied, s_j = s1 * 2^-(j+1) for the j-th extra bit
  (the expected absolute residual of a uniform residual on a cell of width s_{j-1}*2), which makes
  the b-bit code the b most significant bits of the top-width code.
* Residual scales, ``scale_mode = 1``: free, one scale per (row, group) and extra bit, as Eq. 4 and
  Eq. 5 print them.  Eq. 5 picks s_{b_k} to minimise || R X - s Q X ||; without calibration data
  (X proportional to the identity) and with Q = sign(R) the minimiser is the mean absolute residual
  of the group, s_j = mean_G |R|, which is what is stored (rounded to the nearest fp16; the paper
  does not say how scales are stored).  The mean is an fp32 sum in a pinned order (32 strided
  partial sums, then a butterfly) so that the stored scales, and with them every later bit, are
  reproducible bit for bit.  The codes stay nested either way: the bits up to width b do not depend
  on later steps.
* The reconstruction rule printed below Eq. 5 has a garbled summation index; it is read as
  W_hat_{b_k} = W_hat_{b_1} + sum_i s_{b_i} Q_{W_{b_i}}.
* Width lists that skip widths (2,4,8) run every one-bit step internally and expose only the
  listed widths.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

F32 = np.float32


def fp16_round_down(x: np.ndarray) -> np.ndarray:
    """Largest fp16-representable value <= x, returned as fp32."""
    x = np.asarray(x, dtype=F32)
    h = x.astype(np.float16)
    too_big = h.astype(F32) > x
    h = np.where(too_big, np.nextafter(h, np.float16(-np.inf)), h).astype(np.float16)
    return h.astype(F32)


def fp16_round_up(x: np.ndarray) -> np.ndarray:
    """Smallest fp16-representable value >= x, returned as fp32."""
    x = np.asarray(x, dtype=F32)
    h = x.astype(np.float16)
    too_small = h.astype(F32) < x
    h = np.where(too_small, np.nextafter(h, np.float16(np.inf)), h).astype(np.float16)
    return h.astype(F32)


@dataclass
class MWQTensor:
    """Nested code of one weight matrix.

    code : uint8 [rows, cols], the top-width code (``bits[-1]`` significant bits).
    s1   : fp32 [rows, cols/g], base scale (an fp16-representable value).
    lo   : fp32 [rows, cols/g], base offset = -z*s of Eq. 2 (an fp16-representable value).
    s_extra : None (tied residual scales) or fp32 [rows, cols/g, top - b1]: the free scale of every
           extra bit, s_extra[..., j-1] = s_j of Eq. 4 (fp16-representable values).
    """
    code: np.ndarray
    s1: np.ndarray
    lo: np.ndarray
    bits: Tuple[int, ...]
    group_size: int
    s_extra: Optional[np.ndarray] = None

    @property
    def top(self) -> int:
        return self.bits[-1]

    @property
    def b1(self) -> int:
        return self.bits[0]


def check_bits(bits: Sequence[int]) -> None:
    assert len(bits) >= 1 and bits[0] >= 1 and bits[-1] <= 8
    assert all(bits[i] < bits[i + 1] for i in range(len(bits) - 1)), "widths must ascend"


def sum_pinned(a: np.ndarray) -> np.ndarray:
    """fp32 sum over the last axis in the pinned order: partial sum l takes elements l, l+32, ... in
    ascending order, then a butterfly over the 32 partial sums (offsets 16, 8, 4, 2, 1)."""
    a = np.ascontiguousarray(a, dtype=F32)
    n = a.shape[-1]
    if n % 32:
        a = np.concatenate([a, np.zeros(a.shape[:-1] + (32 - n % 32,), dtype=F32)], axis=-1)
    a = a.reshape(a.shape[:-1] + (-1, 32))
    acc = np.zeros(a.shape[:-2] + (32,), dtype=F32)
    for m in range(a.shape[-2]):
        acc = (acc + a[..., m, :]).astype(F32)
    lanes = np.arange(32)
    for off in (16, 8, 4, 2, 1):
        acc = (acc + acc[..., lanes ^ off]).astype(F32)
    return acc[..., 0]


def quantize(W: np.ndarray, bits: Sequence[int], group_size: int, scale_mode: int = 0,
             col_energy: Optional[np.ndarray] = None, return_what: bool = False):
    """MWQ of W [rows, cols] with groups of ``group_size`` along the input (column) axis.

    ``col_energy`` (scale_mode 1 only): per input column i the second moment d_i of the calibration
    activations.  Eq. 5 with the cross-column terms of X X^T dropped is a weighted least-squares fit, whose
    minimiser for Q = sign(R) is s = sum_i d_i |R_i| / sum_i d_i over the group (both sums in the pinned
    order); with equal energies it is the plain mean.  ``return_what``: also return the fp32 reconstruction
    at the top width as the quantizer itself accumulated it (used by the block compensation).

    Step 1 is the per-group asymmetric b1-bit quantization of Eq. 2; steps 2.. are the binary
    residual quantization of Eq. 4, one bit per step up to the top width, with tied scales
    (``scale_mode = 0``) or with the free per-step scale of Eq. 5 (``scale_mode = 1``, see the
    module docstring).  All arithmetic is fp32 with one rounding per operation (numpy does not
    contract a*b+c).
    """
    assert scale_mode in (0, 1)
    check_bits(bits)
    W = np.ascontiguousarray(W, dtype=F32)
    rows, cols = W.shape
    g = group_size
    assert cols % g == 0
    b1, top = bits[0], bits[-1]
    Wg = W.reshape(rows, cols // g, g)

    wmin = Wg.min(axis=2)
    wmax = Wg.max(axis=2)
    lo = fp16_round_down(wmin)
    s1 = fp16_round_up((wmax - lo) / F32(2 ** b1 - 1))
    s1 = np.where(s1 == 0, F32(2.0 ** -14), s1).astype(F32)

    lo_b = lo[:, :, None]
    s1_b = s1[:, :, None]
    # Eq. 2: Q = round(W/s + z) with z = -lo/s, evaluated as round((W - lo)/s)
    Q = np.clip(np.rint((Wg - lo_b) / s1_b), F32(0), F32(2 ** b1 - 1)).astype(F32)
    What = (lo_b + Q * s1_b).astype(F32)              # (Q - z) * s
    R = (Wg - What).astype(F32)
    code = Q.astype(np.int32)
    s_extra = np.zeros((rows, cols // g, top - b1), dtype=F32) if scale_mode == 1 else None
    if col_energy is not None:
        assert scale_mode == 1
        dg = np.ascontiguousarray(col_energy, dtype=F32).reshape(1, cols // g, g)
        den = sum_pinned(dg)                                   # [1, groups]
    for j in range(1, top - b1 + 1):
        if scale_mode == 0:
            s_j = (s1_b * F32(2.0 ** -(j + 1))).astype(F32)   # exact: power-of-two multiple
        elif col_energy is not None:
            # Eq. 5 with per-column activation energies: weighted mean of |R|
            mean_abs = (sum_pinned((np.abs(R) * dg).astype(F32)) / den).astype(F32)
            s_extra[:, :, j - 1] = mean_abs.astype(np.float16).astype(F32)
            s_j = s_extra[:, :, j - 1][:, :, None]
        else:
            # Eq. 5 without calibration data: argmin_s ||R - s sign(R)||^2 = mean |R| over the group
            mean_abs = (sum_pinned(np.abs(R)) / F32(g)).astype(F32)
            s_extra[:, :, j - 1] = mean_abs.astype(np.float16).astype(F32)
            s_j = s_extra[:, :, j - 1][:, :, None]
        bit = R >= 0                                       # Eq. 4, Q in {+1,-1}
        What = (What + np.where(bit, s_j, -s_j)).astype(F32)
        R = (Wg - What).astype(F32)
        code = code * 2 + bit.astype(np.int32)
    assert code.min() >= 0 and code.max() < (1 << top)
    q = MWQTensor(code.reshape(rows, cols).astype(np.uint8), s1, lo, tuple(bits), g, s_extra)
    if return_what:
        return q, What.reshape(rows, cols)
    return q


def quantize_calibrated(W: np.ndarray, bits: Sequence[int], group_size: int, hc: Optional[np.ndarray],
                        col_energy: Optional[np.ndarray] = None) -> MWQTensor:
    """Calibration-aware MWQ (Eq. 3 / Eq. 5 and Algorithm 1) with free per-step scales.

    ``hc``: the upper-triangular Cholesky factor H^c of (2 X X^T + lambda I)^-1 that Algorithm 1 starts from,
    fp32 [cols, cols].  Reading of Algorithm 1 (its printed loop nest is garbled: the level loop never reaches
    K, W is changed inside it, E is divided by an index that is not a block): blocks are the quantization
    groups (gamma = g), taken left to right; a block is quantized at once through all its steps (Eq. 2, then
    Eq. 4 with the scales of Eq. 5) - Section 3.3.1 says that errors are compensated per block, not per
    column -; its error at the top width, column j divided by H^c[j, j], is then taken
    out of all later columns: W[:, later] -= E H^c[block, later].  All of it fp32, one rounding per operation,
    the update as g successive rank-one corrections in ascending column order (so that it is reproducible bit
    for bit).  PARITY UNPINNED as far as that reading goes; what is pinned: with a diagonal H^c nothing is
    propagated and the result is ``quantize(..., scale_mode=1)``; the first block never changes; on correlated
    activations the compensated weights reproduce W X better than the uncompensated ones.
    """
    check_bits(bits)
    W = np.array(W, dtype=F32, copy=True)
    rows, cols = W.shape
    g = group_size
    assert cols % g == 0
    parts = []
    for b in range(0, cols, g):
        ce = None if col_energy is None else np.asarray(col_energy, dtype=F32)[b:b + g]
        q, what = quantize(W[:, b:b + g], bits, g, scale_mode=1, col_energy=ce, return_what=True)
        parts.append(q)
        if hc is not None and b + g < cols:
            hcf = np.asarray(hc, dtype=F32)
            diag = hcf[np.arange(b, b + g), np.arange(b, b + g)]
            E = ((W[:, b:b + g] - what).astype(F32) / diag[None, :]).astype(F32)
            for j in range(g):
                W[:, b + g:] = (W[:, b + g:] - (E[:, j:j + 1] * hcf[b + j, b + g:][None, :]).astype(F32)).astype(F32)
    code = np.concatenate([q.code for q in parts], axis=1)
    s1 = np.concatenate([q.s1 for q in parts], axis=1)
    lo = np.concatenate([q.lo for q in parts], axis=1)
    s_extra = np.concatenate([q.s_extra for q in parts], axis=1)
    return MWQTensor(code, s1, lo, tuple(bits), g, s_extra)


def slice_code(q: MWQTensor, b: int) -> np.ndarray:
    """Code at width b: the b most significant bits of the top-width code (matryoshka nesting)."""
    assert q.b1 <= b <= q.top
    return (q.code >> (q.top - b)).astype(np.uint8)


def dequantize(q: MWQTensor, b: int) -> np.ndarray:
    """fp64 weights at width b by the paper's additive rule (below Eq. 5):
    W_hat_b = (Q_b1 - z) * s_b1 + sum over the extra bits j = 1..b-b1 of s_j * (+1 or -1)."""
    assert q.b1 <= b <= q.top
    rows, cols = q.code.shape
    g = q.group_size
    code = q.code.reshape(rows, cols // g, g).astype(np.int64)
    s1 = q.s1.astype(np.float64)[:, :, None]
    lo = q.lo.astype(np.float64)[:, :, None]
    base = code >> (q.top - q.b1)
    W = lo + base.astype(np.float64) * s1
    for j in range(1, b - q.b1 + 1):
        bit = (code >> (q.top - q.b1 - j)) & 1
        s_j = s1 * 2.0 ** -(j + 1) if q.s_extra is None else q.s_extra[:, :, j - 1].astype(np.float64)[:, :, None]
        W = W + np.where(bit == 1, 1.0, -1.0) * s_j
    return W.reshape(rows, cols)


def dequantize_closed_form(q: MWQTensor, b: int) -> np.ndarray:
    """Same weights from the sliced integer code alone: with q_b = code >> (top-b) and
    s_b = s1 / 2^(b-b1), W_hat_b = (lo - s1/2) + s_b * (q_b + 1/2), the midpoint of cell q_b of a
    uniform grid of 2^b cells.  Used to pin ``dequantize`` (two independent formulas).  Tied scales only."""
    assert q.s_extra is None
    rows, cols = q.code.shape
    g = q.group_size
    qb = slice_code(q, b).reshape(rows, cols // g, g).astype(np.float64)
    s1 = q.s1.astype(np.float64)[:, :, None]
    lo = q.lo.astype(np.float64)[:, :, None]
    sb = s1 / 2.0 ** (b - q.b1)
    return ((lo - s1 / 2) + sb * (qb + 0.5)).reshape(rows, cols)


def segments(bits: Sequence[int]) -> List[Tuple[int, int]]:
    """The nested store as segments: (shift, width) of each segment inside the top-width code.
    Segment 0 holds the b1 base bits; segment j the bits[j]-bits[j-1] bits added next."""
    check_bits(bits)
    top = bits[-1]
    out, prev = [], 0
    for b in bits:
        out.append((top - b, b - prev))
        prev = b
    return out


def segment_values(q: MWQTensor) -> List[np.ndarray]:
    return [((q.code >> sh) & ((1 << w) - 1)).astype(np.uint8) for sh, w in segments(q.bits)]


def segments_read(width_idx: int) -> List[int]:
    """Segments an expert call at ``bits[width_idx]`` reads: all up to and including its own."""
    return list(range(width_idx + 1))


def segment_use_counts(width_idx_of_requests: Sequence[int], n_bits: int) -> List[int]:
    """How many requests on one expert read each segment (Section 3.4's plane-reuse example)."""
    counts = [0] * n_bits
    for k in width_idx_of_requests:
        for j in segments_read(k):
            counts[j] += 1
    return counts


def nested_store_bits_per_weight(bits: Sequence[int]) -> int:
    """Bits stored per weight by the nested store: the top width only, whatever the list is."""
    return sum(w for _, w in segments(bits))
