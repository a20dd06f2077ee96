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


# ---------------------------------------------------------------- free per-level scales (Eq. 4 and Eq. 5, scale_mode = 1)
def test_sum_pinned_is_an_exact_sum_on_integers_and_order_sensitive():
    a = rng.integers(-1000, 1000, size=(5, 7, 96)).astype(F32)
    assert np.array_equal(mwq.sum_pinned(a), a.sum(axis=-1, dtype=np.float64).astype(F32))
    # an input where a plain left-to-right fp32 sum gives another float than the pinned order
    x = np.zeros(64, dtype=F32)
    x[0], x[1], x[33] = F32(2.0 ** 24), F32(1.0), F32(1.0)
    seq = F32(0)
    for v in x:
        seq = F32(seq + v)
    assert seq == F32(2.0 ** 24)                      # each 1.0 is absorbed on its own
    assert mwq.sum_pinned(x) == F32(2.0 ** 24 + 2.0)  # pinned: partial sum 1 holds 1.0 + 1.0, and 2^24 + 2 is exact
    # whatever the order, the result stays within n ulps of the fp64 sum
    y = np.abs(gaussian(3, 256, seed=11))
    assert np.allclose(mwq.sum_pinned(y), y.sum(axis=-1, dtype=np.float64), rtol=1e-6)


def test_free_scales_share_the_base_step_and_keep_the_codes_nested():
    W = gaussian(16, 256, seed=21)
    bits = (2, 3, 4, 8)
    tied = mwq.quantize(W, bits, 64)
    free = mwq.quantize(W, bits, 64, scale_mode=1)
    # Eq. 2 is untouched: base code, scale and offset are those of the tied mode
    assert np.array_equal(free.s1, tied.s1) and np.array_equal(free.lo, tied.lo)
    assert np.array_equal(mwq.slice_code(free, 2), mwq.slice_code(tied, 2))
    # the first residual bit only depends on the sign of the base residual: also shared
    assert np.array_equal(mwq.slice_code(free, 3), mwq.slice_code(tied, 3))
    assert free.s_extra.shape == (16, 4, 6)
    assert np.array_equal(free.s_extra.astype(np.float16).astype(F32), free.s_extra)      # fp16-representable
    # truncated lists give the MSB prefix of the codes and the prefix of the scales
    for n in range(1, len(bits)):
        part = mwq.quantize(W, bits[:n], 64, scale_mode=1)
        assert np.array_equal(part.code, mwq.slice_code(free, bits[n - 1]))
        assert np.array_equal(part.s_extra, free.s_extra[:, :, :bits[n - 1] - 2])


def test_free_scale_is_the_least_squares_scale_of_the_sign_code():
    """Eq. 5 with X = I and Q = sign(R): argmin_s ||R - s Q||^2 = mean |R|.  Brute force: recompute the residual
    before every step from the stored codes and scales, and check that no fp16 neighbour of the stored scale
    (nor any scale of a fine grid) gives a smaller squared error."""
    W = gaussian(6, 128, seed=22)
    bits, g = (2, 8), 32
    q = mwq.quantize(W, bits, g, scale_mode=1)
    Wg = W.reshape(6, 4, g).astype(np.float64)
    code = q.code.reshape(6, 4, g).astype(np.int64)
    What = q.lo.astype(np.float64)[:, :, None] + (code >> 6) * q.s1.astype(np.float64)[:, :, None]
    for j in range(1, 7):
        R = Wg - What
        sign = np.where(((code >> (6 - j)) & 1) == 1, 1.0, -1.0)
        assert np.array_equal(sign, np.where(R >= 0, 1.0, -1.0))            # Eq. 4: Q = sign(R)
        s = q.s_extra[:, :, j - 1].astype(np.float64)
        err = lambda sc: ((R - sc[:, :, None] * sign) ** 2).sum(axis=2)
        best = err(s)
        h = q.s_extra[:, :, j - 1].astype(np.float16)
        for nb in (np.nextafter(h, np.float16(np.inf)), np.nextafter(h, np.float16(-np.inf))):
            assert np.all(best <= err(nb.astype(np.float64)) * (1 + 1e-12))
        # the error is a parabola in the scale with its minimum at mean |R|; the stored scale is that value rounded to
        # fp16, i.e. at most g (2^-11 s)^2 above the minimum: no scale of a fine grid does better than that
        slack = g * (2.0 ** -11 * s) ** 2
        for f in np.linspace(0.0, 3.0, 61):
            assert np.all(best <= err(s * f) + slack)
        assert np.allclose(s, np.abs(R).mean(axis=2), rtol=2.0 ** -10)       # = mean |R| up to fp16 rounding
        What = What + s[:, :, None] * sign


def test_free_scales_never_increase_the_error_and_dequantize_is_additive():
    W = gaussian(8, 256, seed=23)
    q = mwq.quantize(W, (2, 3, 4, 8), 128, scale_mode=1)
    prev = None
    for b in range(2, 9):
        Wb = mwq.dequantize(q, b)
        e = ((Wb - W) ** 2).reshape(8, 2, 128).sum(axis=2)
        if prev is not None:
            assert np.all(e <= prev * (1 + 1e-3))          # each step's scale minimises that step's error (fp16-rounded)
        prev = e
    # additive rule written out for one weight
    r, c, g = 3, 200, 128
    G, top, b1 = c // g, 8, 2
    code = int(q.code[r, c])
    w = float(q.lo[r, G]) + (code >> 6) * float(q.s1[r, G])
    for j in range(1, 7):
        w += (1.0 if (code >> (6 - j)) & 1 else -1.0) * float(q.s_extra[r, G, j - 1])
    assert mwq.dequantize(q, 8)[r, c] == pytest.approx(w, rel=1e-15)


def test_free_scales_approach_the_tied_ones_on_uniform_residuals():
    # weights spread uniformly over the base grid's range: the mean absolute residual of a uniform residual on a cell
    # of width c is c / 4, so s_1 ~ s1 / 4, s_2 ~ s1 / 8, ...: the free scales fall back on the tied ones
    r = np.random.default_rng(24)
    W = r.uniform(-1.0, 1.0, size=(4, 4096)).astype(F32)
    q = mwq.quantize(W, (2, 8), 256, scale_mode=1)
    for j in range(1, 4):
        ratio = q.s_extra[:, :, j - 1] / (q.s1 * 2.0 ** -(j + 1))
        assert np.all(np.abs(ratio - 1.0) < 0.15), (j, ratio.min(), ratio.max())


# ---------------------------------------------------------------- calibration-aware MWQ (Eq. 5 with activation energies, Algorithm 1)
def calib(cols, n=512, seed=0, corr=0.6):
    """Correlated synthetic calibration activations X [cols, n] and the factor Algorithm 1 starts from."""
    import torch
    r = np.random.default_rng(seed)
    base = r.standard_normal((cols, n))
    mix = np.eye(cols) + corr * np.roll(np.eye(cols), 1, axis=1) + 0.3 * corr * np.roll(np.eye(cols), 7, axis=1)
    X = (mix @ base) * (0.5 + r.random((cols, 1)) * 2.0)
    H = 2.0 * X @ X.T / n + 1e-2 * np.eye(cols)
    Hinv = np.linalg.inv(H)
    hc = torch.linalg.cholesky(torch.from_numpy(Hinv), upper=True).numpy().astype(F32)
    return X, hc, (X * X).mean(axis=1).astype(F32)


def test_weighted_scale_is_the_weighted_least_squares_scale():
    W = gaussian(5, 128, seed=31)
    d = (np.random.default_rng(32).random(128) * 3 + 0.1).astype(F32)
    q = mwq.quantize(W, (2, 8), 32, scale_mode=1, col_energy=d)
    Wg = W.reshape(5, 4, 32).astype(np.float64)
    dg = d.reshape(1, 4, 32).astype(np.float64)
    code = q.code.reshape(5, 4, 32).astype(np.int64)
    What = q.lo.astype(np.float64)[:, :, None] + (code >> 6) * q.s1.astype(np.float64)[:, :, None]
    for j in range(1, 7):
        R = Wg - What
        sign = np.where(R >= 0, 1.0, -1.0)
        s = q.s_extra[:, :, j - 1].astype(np.float64)
        err = lambda sc: (dg * (R - sc[:, :, None] * sign) ** 2).sum(axis=2)
        slack = (dg.sum(axis=2)) * (2.0 ** -11 * s) ** 2
        for f in np.linspace(0.0, 3.0, 61):
            assert np.all(err(s) <= err(s * f) + slack)
        assert np.allclose(s, (dg * np.abs(R)).sum(axis=2) / dg.sum(axis=2), rtol=2.0 ** -10)
        What = What + s[:, :, None] * sign
    # equal energies: the plain mean of scale_mode 1, whatever their common value
    a = mwq.quantize(W, (2, 8), 32, scale_mode=1)
    b = mwq.quantize(W, (2, 8), 32, scale_mode=1, col_energy=np.full(128, 4.0, dtype=F32))
    assert np.array_equal(a.code, b.code) and np.array_equal(a.s_extra, b.s_extra)


def test_block_compensation_special_cases_and_effect():
    W = gaussian(48, 256, seed=33)
    bits, g = (2, 3, 4, 8), 64
    plain = mwq.quantize(W, bits, g, scale_mode=1)
    # a diagonal factor propagates nothing: the calibration-free result
    diag = np.diag(np.linspace(0.5, 2.0, 256)).astype(F32)
    q = mwq.quantize_calibrated(W, bits, g, diag)
    assert np.array_equal(q.code, plain.code) and np.array_equal(q.s_extra, plain.s_extra) and np.array_equal(q.s1, plain.s1)
    assert np.array_equal(mwq.quantize_calibrated(W, bits, g, None).code, plain.code)
    # correlated activations: the first block is untouched, later blocks change, and W X is reproduced better at every width
    X, hc, energy = calib(256, seed=34)
    qc = mwq.quantize_calibrated(W, bits, g, hc)
    assert np.array_equal(qc.code[:, :g], plain.code[:, :g]) and not np.array_equal(qc.code[:, g:], plain.code[:, g:])
    ref = W.astype(np.float64) @ X
    for b in (4, 8):
        e_plain = np.linalg.norm(mwq.dequantize(plain, b) @ X - ref)
        e_comp = np.linalg.norm(mwq.dequantize(qc, b) @ X - ref)
        assert e_comp < e_plain, (b, e_comp, e_plain)
    # and with the energies in the scale fit as well it still runs through the same machinery
    qe = mwq.quantize_calibrated(W, bits, g, hc, energy)
    assert qe.code.shape == W.shape and np.array_equal(qe.code[:, :g] >> 6, plain.code[:, :g] >> 6)
