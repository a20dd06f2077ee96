"""Pins for the routing oracle: exact-arithmetic cases, library routines, brute force."""
import numpy as np
import pytest
import scipy.special
import torch

from oracle import routing

F32 = np.float32


def bf16(a):
    return torch.from_numpy(np.asarray(a, dtype=F32)).to(torch.bfloat16).to(torch.float32).numpy()


def test_logits_exact_on_small_integers():
    r = np.random.default_rng(0)
    x = r.integers(-8, 9, size=(5, 96)).astype(F32)
    W = r.integers(-8, 9, size=(7, 96)).astype(F32)
    got = routing.logits_pinned(x, W)
    assert np.array_equal(got, (x.astype(np.int64) @ W.astype(np.int64).T).astype(F32))


def test_logits_close_to_fp64_dot():
    r = np.random.default_rng(1)
    x = bf16(r.standard_normal((9, 1000)))           # d not a multiple of 32
    W = bf16(r.standard_normal((6, 1000)) * 0.02)
    got = routing.logits_pinned(x, W)
    ref = x.astype(np.float64) @ W.astype(np.float64).T
    scale = np.abs(x.astype(np.float64))[:, None, :] * np.abs(W.astype(np.float64))[None, :, :]
    assert np.all(np.abs(got - ref) <= 1e-6 * scale.sum(axis=2) + 1e-12)


def test_logits_summation_order_is_the_pinned_one():
    """Lane 0 sees 2^24, then 1, then -2^24: the strided per-lane order loses the 1 (fp32 spacing at
    2^24 is 2), any order that pairs 2^24 with -2^24 first keeps it.  Lane 1 holds a 3."""
    x = np.zeros((1, 96), dtype=F32)
    W = np.ones((1, 96), dtype=F32)
    x[0, 0], x[0, 32], x[0, 64] = 2.0 ** 24, 1.0, -(2.0 ** 24)
    x[0, 1] = 3.0
    assert routing.logits_pinned(x, W)[0, 0] == F32(3.0)
    # the same numbers in three different lanes survive: lanes 0,1,2 hold 2^24, 1, -2^24; offsets
    # 16, 8, 4 add zeros, offset 2 pairs lane 0 with lane 2 (cancelling), offset 1 adds the 1
    y = np.zeros((1, 96), dtype=F32)
    y[0, 0], y[0, 1], y[0, 2] = 2.0 ** 24, 1.0, -(2.0 ** 24)
    assert routing.logits_pinned(y, W)[0, 0] == F32(1.0)


def test_topk_matches_stable_sort_and_torch():
    r = np.random.default_rng(2)
    logits = r.standard_normal((64, 8)).astype(F32)
    idx = routing.topk_select(logits, 2)
    ref = np.argsort(-logits, axis=1, kind="stable")[:, :2]
    assert np.array_equal(idx, ref.astype(np.int32))
    tv, ti = torch.topk(torch.from_numpy(logits), 2, dim=1)
    assert np.array_equal(idx, ti.numpy().astype(np.int32))


def test_topk_ties_go_to_lower_index():
    logits = np.array([[1.0, 3.0, 3.0, 0.0, 3.0], [0.0, 0.0, 0.0, 0.0, 0.0]], dtype=F32)
    idx = routing.topk_select(logits, 3)
    assert idx.tolist() == [[1, 2, 4], [0, 1, 2]]


@pytest.mark.parametrize("renorm", [False, True])
def test_gate_weights_match_library_softmax(renorm):
    r = np.random.default_rng(3)
    logits = (r.standard_normal((40, 8)) * 3).astype(F32)
    idx = routing.topk_select(logits, 2)
    w = routing.gate_weights(logits, idx, renorm)
    p = scipy.special.softmax(logits.astype(np.float64), axis=1)
    ref = np.take_along_axis(p, idx.astype(np.int64), axis=1)
    if renorm:
        ref = ref / ref.sum(axis=1, keepdims=True)
        assert np.allclose(w.sum(axis=1), 1.0, atol=1e-14)
    assert np.allclose(w, ref, rtol=1e-13, atol=0)
    assert np.all(w[:, 0] >= w[:, 1])               # selection order is by descending logit


def test_grouping_is_a_stable_sort_by_expert_then_width():
    r = np.random.default_rng(4)
    T, k, E, K = 50, 3, 6, 4
    idx = np.stack([r.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    bit_idx = r.integers(0, K, size=(T, k)).astype(np.int8)
    g = routing.group_assignments(idx, bit_idx, E, K)
    keys = (idx.astype(np.int64) * K + bit_idx).reshape(-1)
    assert np.array_equal(g.perm, np.argsort(keys, kind="stable").astype(np.int32))
    assert np.array_equal(np.sort(g.perm), np.arange(T * k))                  # bijection
    assert np.array_equal(g.perm[g.inv_perm], np.arange(T * k))
    assert np.array_equal(g.hist.reshape(-1), np.bincount(keys, minlength=E * K))
    assert np.array_equal(g.group_off, np.concatenate([[0], np.cumsum(g.hist.reshape(-1))]))
    for key in range(E * K):
        seg = g.perm[g.group_off[key]:g.group_off[key + 1]]
        assert np.all(keys[seg] == key) and np.all(np.diff(seg) > 0)         # contiguous, stable


def test_bit_width_choice_argmax_first_wins():
    d, E, K = 64, 3, 4
    x = bf16(np.random.default_rng(5).standard_normal((4, d)))
    Wb = np.zeros((E, K, d), dtype=F32)
    Wb[0, 2] = x[0]                # token 0 on expert 0 -> width index 2
    Wb[1, 1] = x[1]; Wb[1, 3] = x[1]   # exact tie between widths 1 and 3 -> 1
    idx = np.array([[0], [1], [2], [2]], dtype=np.int32)
    out = routing.bit_width_choice(x, bf16(Wb), idx)
    assert out[0, 0] == 2 and out[1, 0] == 1
    assert out[2, 0] == 0 and out[3, 0] == 0      # all-zero logits: lowest width


def test_route_end_to_end_small():
    r = np.random.default_rng(6)
    T, d, E, K, k = 12, 64, 4, 3, 2
    x = bf16(r.standard_normal((T, d)))
    gw = bf16(r.standard_normal((E, d)) * 0.1)
    forced = r.integers(0, K, size=(T, k)).astype(np.int8)
    rt = routing.route(x, E=E, K=K, top_k=k, renormalize=True, gate_w=gw, forced_bit_idx=forced)
    assert np.array_equal(rt.bit_idx, forced)
    rt2 = routing.route(x, E=E, K=K, top_k=k, renormalize=True, logits=rt.logits, forced_bit_idx=forced)
    assert np.array_equal(rt.topk_idx, rt2.topk_idx) and np.array_equal(rt.grouping.perm, rt2.grouping.perm)
    assert rt.grouping.hist.sum() == T * k
