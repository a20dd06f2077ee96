"""Pins for the FFN / combine oracle: library routines, linearity, the INT8 error bound."""
import numpy as np
import pytest
import torch

from oracle import moe, mwq, routing

F32 = np.float32


def bf16(a):
    return torch.from_numpy(np.asarray(a, dtype=F32)).to(torch.bfloat16).to(torch.float32).numpy()


def make_layer(seed, d, F, E, g, bits, n_extra=0):
    r = np.random.default_rng(seed)
    raw = {}
    for e in range(E + n_extra):
        raw[e] = ((r.standard_normal((F, d)) * 0.02).astype(F32),
                  (r.standard_normal((F, d)) * 0.02).astype(F32),
                  (r.standard_normal((d, F)) * 0.02).astype(F32))
    packed = {e: tuple(mwq.quantize(m, bits, g) for m in raw[e]) for e in raw}
    return raw, packed


def test_single_expert_top_width_is_a_dense_swiglu_mlp():
    d, F, g, bits = 64, 128, 32, (2, 4, 8)
    raw, packed = make_layer(0, d, F, 1, g, bits)
    x = bf16(np.random.default_rng(1).standard_normal((5, d)))
    rt = routing.route(x, E=1, K=3, top_k=1, renormalize=True, logits=np.zeros((5, 1), dtype=F32),
                       forced_bit_idx=np.full((5, 1), 2, dtype=np.int8))
    y = moe.moe_layer(x, rt, lambda e: packed[e], bits, 1)
    Wg, Wu, Wd = (torch.from_numpy(mwq.dequantize_closed_form(m, 8)) for m in packed[0])
    xt = torch.from_numpy(x.astype(np.float64))
    ref = (torch.nn.functional.silu(xt @ Wg.T) * (xt @ Wu.T)) @ Wd.T
    got = np.stack([y[t] for t in range(5)])
    assert np.allclose(got, ref.numpy(), rtol=1e-11, atol=1e-14)


def test_each_assignment_uses_its_own_width():
    d, F, g, bits, E = 64, 128, 32, (2, 3, 4, 8), 3
    raw, packed = make_layer(2, d, F, E, g, bits)
    T, k = 6, 2
    x = bf16(np.random.default_rng(3).standard_normal((T, d)))
    r = np.random.default_rng(4)
    logits = r.standard_normal((T, E)).astype(F32)
    forced = r.integers(0, 4, size=(T, k)).astype(np.int8)
    rt = routing.route(x, E=E, K=4, top_k=k, renormalize=True, logits=logits, forced_bit_idx=forced)
    y = moe.moe_layer(x, rt, lambda e: packed[e], bits, E)
    for t in range(T):
        ref = np.zeros(d)
        for s in range(k):
            e, b = int(rt.topk_idx[t, s]), bits[int(rt.bit_idx[t, s])]
            Wg, Wu, Wd = (mwq.dequantize_closed_form(m, b) for m in packed[e])
            ref += rt.topk_w[t, s] * moe.swiglu_ffn(x[t:t + 1].astype(np.float64), Wg, Wu, Wd)[0]
        assert np.allclose(y[t], ref, rtol=1e-10, atol=1e-14)
    # token subset gives the same rows
    sub = moe.moe_layer(x, rt, lambda e: packed[e], bits, E, tokens=[4, 1])
    assert set(sub) == {1, 4}
    assert np.allclose(sub[4], y[4], rtol=1e-12, atol=1e-16) and np.allclose(sub[1], y[1], rtol=1e-12, atol=1e-16)


def test_combine_linearity_and_slot_order():
    d, F, g, bits, E = 32, 64, 32, (2, 4, 8), 4
    raw, packed = make_layer(5, d, F, E, g, bits)
    x = bf16(np.random.default_rng(6).standard_normal((3, d)))
    # k = 1 with weight 1 (renormalised) returns the bare expert output
    logits = np.array([[5, 0, 0, 0], [0, 5, 0, 0], [0, 0, 0, 5]], dtype=F32)
    rt = routing.route(x, E=E, K=3, top_k=1, renormalize=True, logits=logits,
                       forced_bit_idx=np.full((3, 1), 1, dtype=np.int8))
    y = moe.moe_layer(x, rt, lambda e: packed[e], bits, E)
    for t, e in enumerate([0, 1, 3]):
        ref = moe.expert_at_width(x[t:t + 1], packed[e], 4)[0]
        assert np.allclose(y[t], ref, rtol=1e-12)
    # swapping the two slots of every token does not change the output
    rt2 = routing.route(x, E=E, K=3, top_k=2, renormalize=True, logits=logits,
                        forced_bit_idx=np.array([[0, 2]] * 3, dtype=np.int8))
    y2 = moe.moe_layer(x, rt2, lambda e: packed[e], bits, E)
    sw = routing.Routing(rt2.logits, rt2.topk_idx[:, ::-1].copy(), rt2.topk_w[:, ::-1].copy(),
                         rt2.bit_idx[:, ::-1].copy(),
                         routing.group_assignments(rt2.topk_idx[:, ::-1], rt2.bit_idx[:, ::-1], E, 3))
    y3 = moe.moe_layer(x, sw, lambda e: packed[e], bits, E)
    for t in range(3):
        assert np.allclose(y2[t], y3[t], rtol=1e-12, atol=1e-16)


def test_shared_experts_are_added_at_top_width_with_weight_one():
    d, F, g, bits, E = 32, 64, 32, (2, 4, 8), 2
    raw, packed = make_layer(7, d, F, E, g, bits, n_extra=1)
    x = bf16(np.random.default_rng(8).standard_normal((4, d)))
    logits = np.random.default_rng(9).standard_normal((4, E)).astype(F32)
    forced = np.zeros((4, 1), dtype=np.int8)
    rt = routing.route(x, E=E, K=3, top_k=1, renormalize=False, logits=logits, forced_bit_idx=forced)
    y0 = moe.moe_layer(x, rt, lambda e: packed[e], bits, E, n_shared=0)
    y1 = moe.moe_layer(x, rt, lambda e: packed[e], bits, E, n_shared=1)
    sh = moe.expert_at_width(x, packed[E], 8)
    for t in range(4):
        assert np.allclose(y1[t] - y0[t], sh[t], rtol=1e-9, atol=1e-15)


def test_matvec_error_bound_at_every_width():
    """|((W - W_hat_b) x)_r| <= sum_G (s_b/2) sum_{i in G} |x_i| (from |W - W_hat_b| <= s_b/2)."""
    g, bits = 64, (2, 3, 4, 8)
    W = (np.random.default_rng(10).standard_normal((32, 256)) * 0.02).astype(F32)
    x = np.random.default_rng(11).standard_normal(256)
    q = mwq.quantize(W, bits, g)
    absx = np.abs(x).reshape(-1, g).sum(axis=1)
    for b in bits:
        err = np.abs(W.astype(np.float64) @ x - mwq.dequantize(q, b) @ x)
        bound = (q.s1.astype(np.float64) / 2.0 ** (b - 2) / 2 * (1 + 1e-5)) @ absx
        assert np.all(err <= bound + 1e-9)


def test_eight_bit_layer_is_within_int8_error_of_unquantized_layer():
    d, F, g, bits, E, T, k = 256, 512, 64, (2, 4, 8), 4, 16, 2
    raw, packed = make_layer(12, d, F, E, g, bits)
    x = bf16(np.random.default_rng(13).standard_normal((T, d)))
    gw = bf16(np.random.default_rng(14).standard_normal((E, d)) * 0.02)
    errs = {}
    for kk in (0, 1, 2):
        rt = routing.route(x, E=E, K=3, top_k=k, renormalize=True, gate_w=gw,
                           forced_bit_idx=np.full((T, k), kk, dtype=np.int8))
        y = moe.moe_layer(x, rt, lambda e: packed[e], bits, E)
        yq = np.stack([y[t] for t in range(T)])
        yr = moe.unquantized_moe_layer(x, rt, lambda e: raw[e], E)
        errs[kk] = np.sqrt(((yq - yr) ** 2).mean()) / np.sqrt((yr ** 2).mean())
    assert errs[2] < 0.03                      # 8 bit: within the INT8 quantization error
    assert errs[2] < errs[1] / 4 < errs[0] / 8  # 16x finer grid per 4 bits


def test_round_to_bf16_and_rmsnorm_match_torch():
    v = np.random.default_rng(15).standard_normal(5000).astype(F32) * 3
    ref = torch.from_numpy(v).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(moe.round_to_bf16(v), ref)
    x = np.random.default_rng(16).standard_normal((7, 96))
    xt = torch.from_numpy(x)
    ref = xt * torch.rsqrt(xt.pow(2).mean(dim=1, keepdim=True) + 1e-5)
    assert np.allclose(moe.rmsnorm(x), ref.numpy(), rtol=1e-13)


def test_stack_layer_residual():
    x = bf16(np.random.default_rng(17).standard_normal((3, 64))).astype(np.float64)
    out = moe.stack_layer(x, lambda xn: np.zeros_like(xn))
    assert np.array_equal(out, x)
    out2 = moe.stack_layer(x, lambda xn: xn)
    assert np.array_equal(out2, moe.round_to_bf16(x + moe.round_to_bf16(moe.rmsnorm(x)).astype(np.float64)))


def test_oracle_sampled_helper_matches_a_direct_layer_call():
    """The test plumbing that cuts a full-size layer by expert (tests/helpers.oracle_sampled) returns
    what one moe_layer call on the whole batch returns, for two batches sharing the weights, with a
    shared expert, on token subsets and with one or several threads."""
    from paper_2504_15299_b200 import synth
    from tests.helpers import OracleLayer, group_edge_tokens, oracle_sampled
    wl = synth.Workload("t", 64, 128, 4, 2, 32, (2, 3, 4, 8), (0.1, 0.2, 0.4, 0.3), seed=9, n_shared=1)
    K = len(wl.bits)
    jobs = []
    for T, tid in ((7, 11), (19, 12)):
        x = synth.bf16_exact(synth.normal(9, tid, (T, wl.d_model), 1.0)).float().numpy()
        logits = synth.normal(9, tid + 10, (T, wl.n_experts), 1.0).numpy()
        fb = synth.categorical(9, tid + 20, (T, wl.top_k), wl.bit_probs).numpy()
        rt = routing.route(x, E=wl.n_experts, K=K, top_k=wl.top_k, renormalize=True, logits=logits, forced_bit_idx=fb)
        jobs.append((x, rt, group_edge_tokens(rt, wl.top_k, extra=2)))
    ol = OracleLayer(wl)
    for n_threads in (1, 3):
        got = oracle_sampled(wl, jobs, n_threads=n_threads)
        for (x, rt, toks), res in zip(jobs, got):
            ref = moe.moe_layer(x, rt, ol, wl.bits, wl.n_experts, wl.n_shared, tokens=toks)
            assert set(res) == set(ref) == set(toks)
            for t in toks:
                assert np.allclose(res[t], ref[t], rtol=1e-12, atol=1e-15)
    # the edge sample touches the first and the last member of every non-empty group
    x, rt, toks = jobs[1]
    gr = rt.grouping
    for key in range(wl.n_experts * K):
        a0, a1 = gr.group_off[key], gr.group_off[key + 1]
        if a1 > a0:
            assert gr.perm[a0] // wl.top_k in toks and gr.perm[a1 - 1] // wl.top_k in toks


def test_elementwise_metric_sees_small_elements():
    from tests.helpers import elementwise_excess, max_norm_rel_err
    ref = np.array([100.0, 1.0, -1.0, 0.5])
    bad = ref.copy()
    bad[3] += 0.6                                  # 0.6 % of the row maximum: invisible to the max-norm metric
    assert max_norm_rel_err(bad, ref) < 1e-2
    assert elementwise_excess(bad, ref) > 1.0
    assert elementwise_excess(ref * (1 + 2.0 ** -9), ref) < 1.0    # bf16 rounding passes
