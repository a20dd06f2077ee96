"""Pins for the MWQ oracle: closed forms, invariants, textbook special cases, brute force."""
import os

import numpy as np
import pytest

from oracle import mwq

F32 = np.float32
rng = np.random.default_rng(1234)


def gaussian(rows, cols, sigma=0.02, seed=0):
    return (np.random.default_rng(seed).standard_normal((rows, cols)) * sigma).astype(F32)


# ---------------------------------------------------------------- fp16 directed rounding
def test_fp16_directed_rounding_known_values():
    # 0.1 lies between the fp16 neighbours 0.0999755859375 and 0.10003662109375
    assert mwq.fp16_round_down(F32(0.1)) == F32(0.0999755859375)
    assert mwq.fp16_round_up(F32(0.1)) == F32(0.10003662109375)
    assert mwq.fp16_round_down(F32(-0.1)) == F32(-0.10003662109375)
    assert mwq.fp16_round_up(F32(-0.1)) == F32(-0.0999755859375)
    # exactly representable values stay put
    for v in (0.0, 0.5, -0.25, 1024.0, 2.0 ** -14, 2.0 ** -24):
        assert mwq.fp16_round_down(F32(v)) == F32(v) and mwq.fp16_round_up(F32(v)) == F32(v)
    # subnormal fp16 range: spacing 2^-24
    x = F32(2.0 ** -24 * 3.5)
    assert mwq.fp16_round_down(x) == F32(2.0 ** -24 * 3) and mwq.fp16_round_up(x) == F32(2.0 ** -24 * 4)


def test_fp16_directed_rounding_brackets():
    x = (rng.standard_normal(20000) * 0.05).astype(F32)
    d, u = mwq.fp16_round_down(x), mwq.fp16_round_up(x)
    assert np.all(d <= x) and np.all(u >= x)
    assert np.all(d.astype(np.float16).astype(F32) == d) and np.all(u.astype(np.float16).astype(F32) == u)
    # neighbours: nothing representable strictly between d and u
    nxt = np.nextafter(d.astype(np.float16), np.float16(np.inf)).astype(F32)
    assert np.all((u == d) | (u == nxt))


# ---------------------------------------------------------------- nesting
@pytest.mark.parametrize("bits", [(2, 3, 4, 8), (2, 4, 8), (4, 8), (5, 6, 7, 8), (3, 5)])
def test_truncated_list_gives_prefix_codes(bits):
    """Quantizing to a shorter list (same b1) gives exactly the MSB prefix of the longer one:
    the low-width weights are nested inside the high-width weights (Section 3.3.1)."""
    W = gaussian(8, 256, seed=3)
    full = mwq.quantize(W, bits, 64)
    for n in range(1, len(bits)):
        part = mwq.quantize(W, bits[:n], 64)
        assert np.array_equal(part.code, mwq.slice_code(full, bits[n - 1]))
        assert np.array_equal(part.s1, full.s1) and np.array_equal(part.lo, full.lo)


def test_width_list_does_not_change_code_or_storage():
    W = gaussian(4, 128, seed=5)
    a = mwq.quantize(W, (2, 3, 4, 8), 64)
    b = mwq.quantize(W, (2, 4, 8), 64)
    c = mwq.quantize(W, (2, 8), 64)
    assert np.array_equal(a.code, b.code) and np.array_equal(a.code, c.code)
    # the nested store costs the top width only, however many widths are served from it
    assert mwq.nested_store_bits_per_weight((2, 3, 4, 8)) == 8
    assert mwq.nested_store_bits_per_weight((2, 4, 8)) == 8
    assert mwq.nested_store_bits_per_weight((2, 3, 4)) == 4
    assert sum((2, 3, 4)) > 4   # separate INT2+INT3+INT4 copies would cost 9 bits per weight


def test_plane_reuse_example_from_paper():
    path = os.path.join(os.path.dirname(__file__), "golden", "plane_reuse_example.txt")
    rec = {}
    for line in open(path):
        if line.startswith("#") or ":" not in line:
            continue
        k, v = line.split(":")
        rec[k.strip()] = [int(t) for t in v.split()]
    bits = rec["bits"]
    req = [bits.index(b) for b in rec["request_widths"]]
    assert mwq.segment_use_counts(req, len(bits)) == rec["segment_readers"]


# ---------------------------------------------------------------- base step = textbook min-max quantizer
@pytest.mark.parametrize("b1", [2, 4, 8])
def test_base_width_is_textbook_asymmetric_minmax(b1):
    g, rows = 64, 6
    r = np.random.default_rng(7)
    levels = 2 ** b1 - 1
    # group min and (max-min)/levels exactly representable in fp16 => no directed-rounding slack
    W = np.empty((rows, g), dtype=F32)
    for i in range(rows):
        lo = F32(np.float16(-0.05 - 0.01 * i))
        scale = F32(np.float16(2.0 ** -6 * (1 + i / 8.0)))
        w = lo + scale * levels * r.random(g).astype(F32)
        w[0], w[1] = lo, F32(lo + scale * levels)
        w = np.clip(w, lo, F32(lo + scale * levels))
        W[i] = w
    q = mwq.quantize(W, (b1,), g)
    wmin = W.min(axis=1, keepdims=True).astype(np.float64)
    wmax = W.max(axis=1, keepdims=True).astype(np.float64)
    scale = (wmax - wmin) / levels
    ref_code = np.clip(np.rint((W.astype(np.float64) - wmin) / scale), 0, levels)
    # identical except where (W-min)/scale sits within fp32 rounding of a .5 boundary
    frac = np.abs(((W.astype(np.float64) - wmin) / scale) % 1.0 - 0.5)
    safe = frac > 1e-4
    assert safe.mean() > 0.99
    assert np.array_equal(q.code[safe], ref_code[safe].astype(np.uint8))
    ref_deq = wmin + ref_code * scale
    assert np.allclose(mwq.dequantize(q, b1)[safe], ref_deq[safe], rtol=0, atol=1e-7)


# ---------------------------------------------------------------- two dequantization formulas
@pytest.mark.parametrize("bits,g", [((2, 3, 4, 8), 128), ((2, 4, 8), 64), ((5, 6, 7, 8), 32), ((3, 4), 16)])
def test_additive_rule_equals_closed_form(bits, g):
    W = gaussian(16, 4 * g, seed=11)
    q = mwq.quantize(W, bits, g)
    for b in range(bits[0], bits[-1] + 1):
        a = mwq.dequantize(q, b)
        c = mwq.dequantize_closed_form(q, b)
        assert np.max(np.abs(a - c)) <= 1e-15 + 1e-13 * np.max(np.abs(a))


def test_reconstruction_is_additive_over_segments():
    bits, g = (2, 3, 4, 8), 128
    W = gaussian(8, 256, seed=13)
    q = mwq.quantize(W, bits, g)
    segs = mwq.segments(bits)
    vals = mwq.segment_values(q)
    assert segs == [(6, 2), (5, 1), (4, 1), (0, 4)]
    s1 = np.repeat(q.s1.astype(np.float64), g, axis=1)
    lo = np.repeat(q.lo.astype(np.float64), g, axis=1)
    s_top = s1 / 2.0 ** (bits[-1] - bits[0])
    for kk, b in enumerate(bits):
        acc = np.zeros(W.shape)
        for j in range(kk + 1):
            acc += vals[j].astype(np.float64) * 2.0 ** segs[j][0]
        s_b = s1 / 2.0 ** (b - bits[0])
        recon = (lo - s1 / 2 + s_b / 2) + s_top * acc
        assert np.allclose(recon, mwq.dequantize(q, b), rtol=0, atol=1e-12)
        # and the code rebuilt from the segments read at this width is the sliced code
        code = np.zeros(W.shape, dtype=np.int64)
        for j in range(kk + 1):
            code |= vals[j].astype(np.int64) << segs[j][0]
        assert np.array_equal(code >> (8 - b), mwq.slice_code(q, b))


# ---------------------------------------------------------------- error bound
@pytest.mark.parametrize("bits", [(2, 3, 4, 8), (2, 4, 8), (4, 8)])
def test_error_bound_halves_per_bit(bits):
    g = 128
    W = gaussian(64, 512, seed=17)
    q = mwq.quantize(W, bits, g)
    s1 = np.repeat(q.s1.astype(np.float64), g, axis=1)
    prev_rms = None
    for b in range(bits[0], bits[-1] + 1):
        err = np.abs(W.astype(np.float64) - mwq.dequantize(q, b))
        s_b = s1 / 2.0 ** (b - bits[0])
        assert np.all(err <= s_b / 2 * (1 + 1e-5) + 1e-9), f"width {b}"
        rms = np.sqrt((err ** 2).mean())
        if prev_rms is not None:
            assert 0.4 < rms / prev_rms < 0.6       # one more bit halves the error
        prev_rms = rms


def test_zero_and_constant_groups():
    W = np.zeros((2, 128), dtype=F32)
    W[1] = F32(0.03125)
    q = mwq.quantize(W, (2, 4, 8), 64)
    assert np.all(q.s1 == F32(2.0 ** -14))
    assert np.max(np.abs(mwq.dequantize(q, 8) - W)) <= 2.0 ** -14


# ---------------------------------------------------------------- brute force on tiny groups
def _reconstruction_points(lo, s1, b1, top):
    """All 2^top reconstruction points, built bit by bit from the paper's additive rule with plain
    python floats (independent of the vectorised oracle)."""
    pts = []
    for code in range(1 << top):
        base = code >> (top - b1)
        v = float(lo) + base * float(s1)
        for j in range(1, top - b1 + 1):
            bit = (code >> (top - b1 - j)) & 1
            v += (1.0 if bit else -1.0) * float(s1) * 2.0 ** -(j + 1)
        pts.append(v)
    return np.array(pts)


@pytest.mark.parametrize("bits", [(2, 3, 4, 8), (3, 6), (1, 2, 3)])
def test_greedy_residual_code_is_nearest_point(bits):
    g = 8
    W = gaussian(12, g, seed=19)
    q = mwq.quantize(W, bits, g)
    for r in range(W.shape[0]):
        pts = _reconstruction_points(q.lo[r, 0], q.s1[r, 0], bits[0], bits[-1])
        assert np.all(np.diff(pts) > 0)             # codes are ordered like their values
        for i in range(g):
            d = np.abs(pts - float(W[r, i]))
            chosen = int(q.code[r, i])
            assert d[chosen] <= d.min() + 1e-9 * float(q.s1[r, 0]) + 1e-12


# ---------------------------------------------------------------- exact round trip on constructed inputs
@pytest.mark.parametrize("bits", [(2, 3, 4, 8), (2, 4, 8)])
def test_round_trip_is_exact_on_grid_inputs(bits):
    """Weights placed exactly on 8-bit reconstruction points come back exactly, and every lower
    width returns the MSB prefix of the chosen code."""
    b1, top, g = bits[0], bits[-1], 64
    s1 = 2.0 ** -5
    lo = -0.0625
    s_top = s1 / 2 ** (top - b1)
    r = np.random.default_rng(23)
    # reconstruction points inside [lo, lo + (2^b1 - 1) s1]: the outer half cells lie beyond the
    # group minimum / maximum and can never be chosen
    half = 1 << (top - b1 - 1)
    codes = r.integers(half, (1 << top) - half, size=(5, g))
    W = (lo - s1 / 2 + s_top * (codes + 0.5)).astype(F32)
    # two anchors fix the group minimum and maximum (they sit on cell edges)
    W[:, 0] = lo
    W[:, 1] = lo + (2 ** b1 - 1) * s1
    q = mwq.quantize(W, bits, g)
    assert np.all(q.s1 == F32(s1)) and np.all(q.lo == F32(lo))
    assert np.array_equal(q.code[:, 2:], codes[:, 2:].astype(np.uint8))
    assert np.array_equal(mwq.dequantize(q, top)[:, 2:], W[:, 2:].astype(np.float64))
    for b in bits:
        assert np.array_equal(mwq.slice_code(q, b)[:, 2:], (codes[:, 2:] >> (top - b)).astype(np.uint8))
    # code-level round trip: a reconstruction point re-quantizes to its own cell
    deq = mwq.dequantize(q, top)
    cell = np.floor((deq - (lo - s1 / 2)) / s_top).astype(np.int64)
    assert np.array_equal(cell, q.code.astype(np.int64))


def test_code_round_trip_on_random_weights():
    bits, g = (2, 3, 4, 8), 128
    W = gaussian(32, 256, seed=29)
    q = mwq.quantize(W, bits, g)
    s1 = np.repeat(q.s1.astype(np.float64), g, axis=1)
    lo = np.repeat(q.lo.astype(np.float64), g, axis=1)
    for b in bits:
        s_b = s1 / 2.0 ** (b - 2)
        cell = np.floor((mwq.dequantize(q, b) - (lo - s1 / 2)) / s_b).astype(np.int64)
        assert np.array_equal(cell, mwq.slice_code(q, b).astype(np.int64))
