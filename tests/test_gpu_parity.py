"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Integer work (codes, routing indices, widths, permutation) is compared bit for bit; layer
outputs within 1e-2 of the row's largest magnitude (fp32 accumulation, bf16 output)."""
import numpy as np
import pytest
import torch

from paper_2504_15299_b200 import synth
from tests.helpers import OracleLayer, check_rows, gpu_layer, max_norm_rel_err, np_f32

pytestmark = pytest.mark.gpu

TOL = 1e-2


@pytest.fixture(scope="module")
def B():
    from paper_2504_15299_b200 import binding, build
    build.build_library()
    binding.lib()
    return binding


def oracle_mods():
    from oracle import moe, mwq, routing
    return mwq, routing, moe


# ------------------------------------------------------------------ pack / unpack
@pytest.mark.parametrize("bits,g,rows,cols", [
    ((2, 4, 8), 64, 512, 256), ((2, 3, 4, 8), 128, 256, 512), ((2, 3, 4), 128, 100, 256),
    ((5, 6, 7, 8), 32, 64, 96), ((3, 5), 64, 130, 128), ((8,), 256, 64, 512), ((1, 2, 3), 32, 70, 64),
    ((4, 8), 128, 192, 1408),
])
def test_pack_codes_bit_exact(B, bits, g, rows, cols):
    mwq, _, _ = oracle_mods()
    cfg = B.Config(cols, cols, 2, 1, g, bits)
    W = synth.normal(11, 5, (rows, cols), 0.02, "cuda")
    blob = B.pack_mwq(cfg, W)
    q = mwq.quantize(np_f32(W), bits, g)
    for b in range(bits[0], bits[-1] + 1):
        codes, s1, lo = B.unpack_codes(cfg, blob, rows, cols, b)
        assert np.array_equal(codes.cpu().numpy(), mwq.slice_code(q, b)), f"width {b}"
    assert np.array_equal(np_f32(s1), q.s1) and np.array_equal(np_f32(lo), q.lo)


def test_pack_degenerate_groups(B):
    mwq, _, _ = oracle_mods()
    cfg = B.Config(128, 128, 2, 1, 64, (2, 4, 8))
    W = torch.zeros((64, 128), device="cuda")
    W[1] = 0.03125
    W[2, :64] = torch.linspace(-1, 1, 64, device="cuda")
    W[3] = synth.normal(1, 1, (1, 128), 1e-6, "cuda")[0]          # tiny range: subnormal fp16 scale
    blob = B.pack_mwq(cfg, W)
    q = mwq.quantize(np_f32(W), (2, 4, 8), 64)
    codes, s1, lo = B.unpack_codes(cfg, blob, 64, 128, 8)
    assert np.array_equal(codes.cpu().numpy(), q.code)
    assert np.array_equal(np_f32(s1), q.s1) and np.array_equal(np_f32(lo), q.lo)


def test_pack_mixtral_matrix_sampled_rows(B):
    """Full-size expert matrix (14336 x 4096, g = 128): the oracle regenerates and quantizes sampled
    rows (first, last, tile edges, random) and every code, scale and offset of those rows must match."""
    mwq, _, _ = oracle_mods()
    wl = synth.WORKLOADS["mixtral_decode"]
    cfg = B.Config.from_workload(wl)
    rows, cols = synth.expert_matrix_shape(wl, 0)
    W = synth.expert_matrix(wl, 3, 0, device="cuda")
    blob = B.pack_mwq(cfg, W)
    del W
    r = np.random.default_rng(0)
    sample = sorted(set([0, 63, 64, 127, 128, rows - 1, rows - 64] + r.integers(0, rows, 40).tolist()))
    Wr = np_f32(synth.expert_matrix(wl, 3, 0, rows=torch.tensor(sample)))
    q = mwq.quantize(Wr, wl.bits, wl.group_size)
    for b in wl.bits:
        codes, s1, lo = B.unpack_codes(cfg, blob, rows, cols, b)
        assert np.array_equal(codes[sample].cpu().numpy(), mwq.slice_code(q, b))
    assert np.array_equal(np_f32(s1[sample]), q.s1) and np.array_equal(np_f32(lo[sample]), q.lo)


# ------------------------------------------------------------------ routing
def check_route(B, cfg, x, *, gate_w=None, logits=None, bit_w=None, forced=None):
    _, routing, _ = oracle_mods()
    K = len(cfg.bits)
    r = B.route(cfg, x, gate_w=gate_w, logits=logits, bit_w=bit_w, forced_bit_idx=forced)
    torch.cuda.synchronize()
    ref = routing.route(np_f32(x), E=cfg.n_experts, K=K, top_k=cfg.top_k, renormalize=bool(cfg.renormalize),
                        gate_w=None if gate_w is None else np_f32(gate_w),
                        logits=None if logits is None else np_f32(logits),
                        bit_w=None if bit_w is None else np_f32(bit_w),
                        forced_bit_idx=None if forced is None else forced.cpu().numpy())
    assert np.array_equal(r.topk_idx.cpu().numpy(), ref.topk_idx)
    assert np.array_equal(r.bit_idx.cpu().numpy(), ref.bit_idx)
    assert np.array_equal(r.perm.cpu().numpy(), ref.grouping.perm)
    assert np.array_equal(r.inv_perm.cpu().numpy(), ref.grouping.inv_perm)
    assert np.array_equal(r.group_off.cpu().numpy(), ref.grouping.group_off)
    assert np.allclose(r.topk_w.cpu().numpy(), ref.topk_w, rtol=1e-5, atol=1e-7)
    assert int(r.device_status.item()) == 0
    return r, ref


@pytest.mark.parametrize("name,T", [("tiny", 16), ("mixtral_decode", 1), ("mixtral_decode", 64),
                                    ("finegrained", 256)])
def test_route_from_gate_weights(B, name, T):
    wl = synth.WORKLOADS[name]
    cfg = B.Config.from_workload(wl)
    x = synth.tokens_bf16(wl, T, "cuda")
    check_route(B, cfg, x, gate_w=synth.gate_weight_bf16(wl, "cuda"), forced=synth.forced_bit_idx(wl, T, "cuda"))


def test_route_from_supplied_logits_prefill(B):
    wl = synth.WORKLOADS["mixtral_prefill"]
    cfg = B.Config.from_workload(wl)
    T = 2048
    x = synth.tokens_bf16(wl, T, "cuda")
    r, ref = check_route(B, cfg, x, logits=synth.zipf_logits(wl, T, "cuda"),
                         forced=synth.forced_bit_idx(wl, T, "cuda"))
    load = ref.grouping.hist.sum(axis=1)
    assert load[0] > 2 * load[-1]                       # the Zipf prior skews the expert loads


def test_route_learned_bit_widths_and_no_renormalize(B):
    wl = synth.WORKLOADS["mixtral_stack"]
    cfg = B.Config.from_workload(wl)
    cfg.renormalize = 0
    x = synth.tokens_bf16(wl, 16, "cuda")
    r, ref = check_route(B, cfg, x, gate_w=synth.gate_weight_bf16(wl, "cuda"),
                         bit_w=synth.bit_router_weight_bf16(wl, "cuda"))
    assert len(set(ref.bit_idx.reshape(-1).tolist())) > 1


def test_route_ties_and_empty_groups(B):
    cfg = B.Config(64, 64, 8, 3, 32, (2, 4, 8))
    T = 5
    x = synth.tokens_bf16(synth.WORKLOADS["tiny"], T, "cuda")[:, :64].contiguous()
    logits = torch.zeros((T, 8), device="cuda")
    logits[1, 5] = logits[1, 2] = 1.0
    logits[2] = torch.tensor([0, 1, 1, 1, 1, 0, 0, 0.0])
    forced = torch.zeros((T, 3), dtype=torch.int8, device="cuda")
    r, ref = check_route(B, cfg, x, logits=logits, forced=forced)
    assert r.topk_idx[0].tolist() == [0, 1, 2] and r.topk_idx[1].tolist() == [2, 5, 0]
    assert r.topk_idx[2].tolist() == [1, 2, 3]


def test_route_flags_nonfinite_logits_and_bad_width_index(B):
    cfg = B.Config(64, 64, 4, 2, 32, (2, 4, 8))
    x = torch.zeros((2, 64), dtype=torch.bfloat16, device="cuda")
    logits = torch.zeros((2, 4), device="cuda")
    logits[1, 2] = float("nan")
    forced = torch.zeros((2, 2), dtype=torch.int8, device="cuda")
    forced[0, 1] = 7
    r = B.route(cfg, x, logits=logits, forced_bit_idx=forced)
    torch.cuda.synchronize()
    st = int(r.device_status.item())
    assert st & B.DEV_NONFINITE and st & B.DEV_BAD_INDEX
    assert int(r.group_off[-1].item()) == 4 and sorted(r.perm.tolist()) == [0, 1, 2, 3]


# ------------------------------------------------------------------ whole layer
def run_layer(B, cfg, wl, T, *, tokens=None, kernel_path=None, blobs=None):
    _, routing, moe = oracle_mods()
    if kernel_path is not None:
        cfg.kernel_path = kernel_path
    x = synth.tokens_bf16(wl, T, "cuda")
    kw = {}
    okw = {}
    if wl.zipf_logits:
        kw["logits"] = synth.zipf_logits(wl, T, "cuda")
        okw["logits"] = np_f32(kw["logits"])
    else:
        kw["gate_w"] = synth.gate_weight_bf16(wl, "cuda")
        okw["gate_w"] = np_f32(kw["gate_w"])
    if wl.learned_bits:
        kw["bit_w"] = synth.bit_router_weight_bf16(wl, "cuda")
        okw["bit_w"] = np_f32(kw["bit_w"])
    else:
        kw["forced_bit_idx"] = synth.forced_bit_idx(wl, T, "cuda")
        okw["forced_bit_idx"] = kw["forced_bit_idx"].cpu().numpy()
    if blobs is None:
        blobs = gpu_layer(B, cfg, wl)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = B.moe_forward(cfg, x, blobs, device_status=status, **kw)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rt = routing.route(np_f32(x), E=wl.n_experts, K=len(wl.bits), top_k=wl.top_k,
                       renormalize=bool(cfg.renormalize), **okw)
    ol = OracleLayer(wl)
    ref = moe.moe_layer(np_f32(x), rt, ol, wl.bits, wl.n_experts, wl.n_shared, tokens=tokens)
    yg = np_f32(y)
    errs = {t: max_norm_rel_err(yg[t], ref[t]) for t in ref}
    return errs, y, blobs


@pytest.mark.parametrize("path", [1, 2])
def test_layer_tiny(B, path):
    wl = synth.WORKLOADS["tiny"]
    errs, _, _ = run_layer(B, B.Config.from_workload(wl), wl, 16, kernel_path=path)
    assert len(errs) == 16 and max(errs.values()) < TOL, errs


def test_layer_finegrained_with_shared_experts_sampled_tokens_cuda_core_path(B):
    # (the tensor-core path is checked on all 256 tokens in test_gpu_parity_configs.py)
    wl = synth.WORKLOADS["finegrained"]
    errs, _, _ = run_layer(B, B.Config.from_workload(wl), wl, 256, tokens=[0, 100, 255], kernel_path=1)
    assert max(errs.values()) < TOL, errs


def cross_check_paths(B, wl, T, blobs=None):
    """Tensor-core path against the CUDA-core path on the same device inputs (all tokens)."""
    x = synth.tokens_bf16(wl, T, "cuda")
    kw = {"forced_bit_idx": synth.forced_bit_idx(wl, T, "cuda")}
    if wl.zipf_logits:
        kw["logits"] = synth.zipf_logits(wl, T, "cuda")
    else:
        kw["gate_w"] = synth.gate_weight_bf16(wl, "cuda")
    cfg_cc = B.Config.from_workload(wl, kernel_path=1)
    cfg_tc = B.Config.from_workload(wl, kernel_path=2)
    if blobs is None:
        blobs = gpu_layer(B, cfg_cc, wl)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    y_cc = B.moe_forward(cfg_cc, x, blobs, device_status=st, **kw).float()
    y_tc = B.moe_forward(cfg_tc, x, blobs, device_status=st, **kw).float()
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    err = (y_cc - y_tc).abs().amax(dim=1) / y_cc.abs().amax(dim=1)
    return float(err.max().item()), blobs


@pytest.fixture(scope="module")
def mixtral_blobs(B):
    wl = synth.WORKLOADS["mixtral_decode"]
    return gpu_layer(B, B.Config.from_workload(wl), wl)


@pytest.mark.parametrize("T", [1, 8, 32, 64])
def test_mixtral_decode_tensor_path_matches_cuda_core_path(B, mixtral_blobs, T):
    wl = synth.WORKLOADS["mixtral_decode"]
    err, _ = cross_check_paths(B, wl, T, mixtral_blobs)
    assert err < TOL, err


def test_layer_empty_batch_is_a_noop(B):
    wl = synth.WORKLOADS["tiny"]
    cfg = B.Config.from_workload(wl)
    x = torch.empty((0, wl.d_model), dtype=torch.bfloat16, device="cuda")
    y = B.moe_forward(cfg, x, [x] * 12, gate_w=synth.gate_weight_bf16(wl, "cuda"),
                      forced_bit_idx=torch.empty((0, 2), dtype=torch.int8, device="cuda"))
    assert y.shape == (0, wl.d_model)


def test_layer_with_precomputed_routing_matches_internal_routing(B):
    wl = synth.WORKLOADS["tiny"]
    cfg = B.Config.from_workload(wl, kernel_path=1)
    x = synth.tokens_bf16(wl, 16, "cuda")
    gw = synth.gate_weight_bf16(wl, "cuda")
    fb = synth.forced_bit_idx(wl, 16, "cuda")
    blobs = gpu_layer(B, cfg, wl)
    y1 = B.moe_forward(cfg, x, blobs, gate_w=gw, forced_bit_idx=fb)
    pre = B.route(cfg, x, gate_w=gw, forced_bit_idx=fb)
    y2 = B.moe_forward(cfg, x, blobs, pre=pre)
    torch.cuda.synchronize()
    assert torch.equal(y1, y2)


def test_stack_layer_tiny(B):
    _, routing, moe = oracle_mods()
    wl = synth.WORKLOADS["tiny"]
    cfg = B.Config.from_workload(wl, kernel_path=1)
    x = synth.tokens_bf16(wl, 16, "cuda")
    x0 = np_f32(x).astype(np.float64)
    gw = synth.gate_weight_bf16(wl, "cuda")
    bw = bit_w = synth.bit_router_weight_bf16(wl, "cuda")
    blobs = gpu_layer(B, cfg, wl)
    xn = torch.empty_like(x)
    B.stack_layer(cfg, x, xn, blobs, gate_w=gw, bit_w=bw)
    torch.cuda.synchronize()
    ol = OracleLayer(wl)

    def moe_of(xnorm):
        rt = routing.route(xnorm.astype(np.float32), E=wl.n_experts, K=len(wl.bits), top_k=wl.top_k,
                           renormalize=True, gate_w=np_f32(gw), bit_w=np_f32(bw))
        out = moe.moe_layer(xnorm, rt, ol, wl.bits, wl.n_experts)
        return np.stack([out[t] for t in range(16)])

    ref = moe.stack_layer(x0, moe_of)
    assert np.array_equal(np_f32(xn), moe.round_to_bf16(moe.rmsnorm(x0)))
    for t in range(16):
        assert max_norm_rel_err(np_f32(x)[t], ref[t]) < TOL


# ------------------------------------------------------------------ prefill (grouped dequant-GEMM) and the stack
def test_mixtral_prefill_tensor_path_matches_cuda_core_path(B, mixtral_blobs):
    """T = 2048 with Zipf-skewed expert loads: the grouped dequant-GEMM (one tile per width, units of up to
    128 tokens, heavy experts split over many units) against the CUDA-core path on every token."""
    wl = synth.WORKLOADS["mixtral_prefill"]
    err, _ = cross_check_paths(B, wl, 2048, mixtral_blobs)
    assert err < TOL, err


# ------------------------------------------------------------------ other width lists, group sizes, loads
def small_layer_case(B, *, d, F, E, k, g, bits, T, n_shared=0, probs=None, seed=21, one_expert=False,
                     token_scales=None, outlier=None, scale_mode=0):
    """Random small layer through the tensor-core path, the CUDA-core path and the oracle."""
    _, routing, moe = oracle_mods()
    from oracle import mwq
    K = len(bits)
    cfg_tc = B.Config(d, F, E, k, g, tuple(bits), n_shared=n_shared, kernel_path=0, scale_mode=scale_mode)
    cfg_cc = B.Config(d, F, E, k, g, tuple(bits), n_shared=n_shared, kernel_path=1, scale_mode=scale_mode)
    raw = {}
    blobs = []
    for e in range(E + n_shared):
        mats = []
        for m in range(3):
            shape = (F, d) if m < 2 else (d, F)
            W = synth.normal(seed, 100 + 3 * e + m, shape, 0.02, "cuda")
            mats.append(np_f32(W))
            blobs.append(B.pack_mwq(cfg_tc, W))
        raw[e] = mats
    x = synth.normal(seed, 1, (T, d), 1.0, "cuda")
    if token_scales is not None:       # per-token magnitudes (0 = an all-zero token)
        x = x * torch.tensor(token_scales, dtype=x.dtype, device="cuda")[:, None]
    if outlier is not None:            # (token, element, value): one element far above the rest of its token
        x[outlier[0], outlier[1]] = outlier[2]
    x = synth.bf16_exact(x)
    logits = synth.normal(seed, 5, (T, E), 1.0, "cuda")
    if one_expert:
        logits[:, 0] += 100.0          # every token picks expert 0 first: units beyond n_cap
    fb = synth.categorical(seed, 4, (T, k), probs or [1.0 / K] * K, "cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    y_tc = B.moe_forward(cfg_tc, x, blobs, logits=logits, forced_bit_idx=fb, device_status=st)
    y_cc = B.moe_forward(cfg_cc, x, blobs, logits=logits, forced_bit_idx=fb, device_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    a, b = y_cc.float(), y_tc.float()
    cross = float(((a - b).abs().amax(dim=1) / a.abs().amax(dim=1).clamp_min(1e-30)).max().item())
    rt = routing.route(np_f32(x), E=E, K=K, top_k=k, renormalize=True, logits=np_f32(logits),
                       forced_bit_idx=fb.cpu().numpy())
    packed = {}

    def get(e):
        if e not in packed:
            packed[e] = tuple(mwq.quantize(W, bits, g, scale_mode) for W in raw[e])
        return packed[e]

    toks = sorted(set([0, T // 2, T - 1]))
    ref = moe.moe_layer(np_f32(x), rt, get, bits, E, n_shared, tokens=toks)
    if token_scales is not None:
        toks = list(range(T))
        ref = moe.moe_layer(np_f32(x), rt, get, bits, E, n_shared, tokens=toks)
    # both metrics: max-norm relative error per token, and the element-wise bound |dy| <= 1e-2 |y| + 1e-2 rms(y)
    # (an all-zero token must come out as exact zeros)
    err, excess = check_rows(np_f32(y_tc), {t: ref[t] for t in toks}, TOL)
    assert excess <= 1.0, excess
    return cross, err


@pytest.mark.parametrize("bits,g", [((2, 3, 4), 128), ((4, 8), 128), ((8,), 64), ((1, 2, 3, 4, 5, 6, 7, 8), 128),
                                    ((3, 5), 64), ((2, 8), 128), ((5, 6, 7, 8), 64), ((5, 6, 7, 8), 128),
                                    ((2, 4, 8), 128), ((2, 3, 4, 8), 64)])
def test_other_width_lists_on_the_tensor_core_paths(B, bits, g):
    cross, err = small_layer_case(B, d=256, F=384, E=4, k=2, g=g, bits=bits, T=24)
    assert cross < TOL and err < TOL, (cross, err)


@pytest.mark.parametrize("bits,g,T", [((2, 3, 4, 8), 128, 24), ((2, 4, 8), 128, 20), ((5, 6, 7, 8), 128, 24),
                                      ((2, 3, 4), 64, 22)])
def test_few_tokens_per_expert_on_average_but_one_crowded_expert(B, bits, g, T):
    # at most 12 tokens per expert on average: the decode kernel runs with ONE fold warpgroup, which must then fold
    # every token block of a full unit (expert 0 gets all T tokens: more than four blocks of four slots)
    cross, err = small_layer_case(B, d=256, F=256, E=4, k=2, g=g, bits=bits, T=T, one_expert=True)
    assert cross < TOL and err < TOL, (cross, err)


def test_all_tokens_on_one_expert_and_shared_experts(B):
    # 80 tokens all choose expert 0 (units beyond the per-unit token cap), one shared expert on top
    cross, err = small_layer_case(B, d=256, F=256, E=4, k=2, g=128, bits=(2, 3, 4, 8), T=80, n_shared=1,
                                  one_expert=True)
    assert cross < TOL and err < TOL, (cross, err)


def test_prefill_sized_load_small_shape(B):
    # 400 tokens on 2 experts: the grouped dequant-GEMM path (more than 24 tokens per expert)
    cross, err = small_layer_case(B, d=256, F=256, E=2, k=1, g=128, bits=(2, 3, 4, 8), T=400,
                                  probs=[0.1, 0.2, 0.4, 0.3])
    assert cross < TOL and err < TOL, (cross, err)


def test_decode_kernel_per_token_activation_scaling(B):
    # the decode kernel quantises every token against its own largest element: tokens of very different
    # magnitude, an all-zero token and a token with one element 100 times above the rest in one batch
    scales = [1.0, 1e-3, 1e3, 0.0, 1.0, 37.5, 2.0 ** -10, 1.0, 5.0]
    cross, err = small_layer_case(B, d=256, F=384, E=2, k=2, g=128, bits=(2, 3, 4, 8), T=9, token_scales=scales,
                                  outlier=(4, 17, 100.0))
    assert err < TOL, err


def test_decode_kernel_flags_nonfinite_activations(B):
    # a NaN in one token: the call is flagged, that token comes out as zeros, the others are untouched
    d, F, E, k, g, bits, T = 256, 256, 2, 1, 128, (2, 4, 8), 6
    cfg = B.Config(d, F, E, k, g, bits)
    blobs = [B.pack_mwq(cfg, synth.normal(31, 100 + i, (F, d) if i % 3 < 2 else (d, F), 0.02, "cuda"))
             for i in range(3 * E)]
    x = synth.bf16_exact(synth.normal(31, 1, (T, d), 1.0, "cuda"))
    logits = synth.normal(31, 5, (T, E), 1.0, "cuda")
    fb = synth.categorical(31, 4, (T, k), [0.3, 0.3, 0.4], "cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    y_clean = B.moe_forward(cfg, x, blobs, logits=logits, forced_bit_idx=fb, device_status=st).clone()
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    x_bad = x.clone()
    x_bad[2, 5] = float("nan")
    x_bad[4, 7] = float("inf")
    y_bad = B.moe_forward(cfg, x_bad, blobs, logits=logits, forced_bit_idx=fb, device_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) & 1                      # D2MOE_DEV_NONFINITE
    keep = [0, 1, 3, 5]
    assert torch.equal(y_bad[keep], y_clean[keep])
    assert float(y_bad[[2, 4]].float().abs().max().item()) == 0.0


def test_workspace_sized_for_a_larger_batch_serves_smaller_ones(B):
    # one workspace sized for 300 tokens (grouped-GEMM kernel) also serves 1 and 16 tokens (decode kernel)
    wl = synth.WORKLOADS["tiny"]
    cfg = B.Config.from_workload(wl)
    blobs = gpu_layer(B, cfg, wl)
    gw = synth.gate_weight_bf16(wl, "cuda")
    ws = torch.empty(B.workspace_bytes(cfg, 300), dtype=torch.uint8, device="cuda")
    for T in (300, 16, 1):
        x = synth.tokens_bf16(wl, T, "cuda")
        fb = synth.forced_bit_idx(wl, T, "cuda")
        y_shared = B.moe_forward(cfg, x, blobs, gate_w=gw, forced_bit_idx=fb, workspace=ws).clone()
        y_own = B.moe_forward(cfg, x, blobs, gate_w=gw, forced_bit_idx=fb)
        torch.cuda.synchronize()
        assert torch.equal(y_shared, y_own)


@pytest.mark.parametrize("case", [
    dict(d=512, F=512, E=128, k=8, g=128, bits=(2, 4, 8), T=64, n_shared=2),        # many experts, few tokens each
    dict(d=256, F=384, E=4, k=2, g=128, bits=(1, 2, 3, 4, 5, 6, 7, 8), T=700),      # eight widths, grouped-GEMM kernel
    dict(d=256, F=256, E=2, k=2, g=64, bits=(2, 4, 8), T=3000),                     # many units per expert, g = 64
    dict(d=384, F=640, E=16, k=4, g=128, bits=(5, 6, 7, 8), T=200, n_shared=1),     # 50 tokens per expert: decode kernel, several units
    dict(d=128, F=128, E=256, k=8, g=128, bits=(2, 4, 8), T=160, n_shared=2),       # more units (266) than threads order at once
])
def test_stress_shapes(B, case):
    cross, err = small_layer_case(B, **case)
    assert cross < TOL and err < TOL, (cross, err)


def test_dense_ffn_single_expert(B):
    # E = 1, k = 1: a dense gated FFN read at a per-token width (the method applied to a dense model)
    cross, err = small_layer_case(B, d=384, F=512, E=1, k=1, g=128, bits=(2, 3, 4, 8), T=20)
    assert cross < TOL and err < TOL, (cross, err)


def test_single_token_and_single_width(B):
    cross, err = small_layer_case(B, d=128, F=128, E=2, k=1, g=64, bits=(2, 4, 8), T=1, probs=[0, 0, 1.0])
    assert cross < TOL and err < TOL, (cross, err)


@pytest.mark.parametrize("d,F,g", [(192, 256, 64), (256, 160, 32), (512, 512, 256)])
def test_shapes_outside_the_tensor_core_path_use_the_cuda_core_path(B, d, F, g):
    # d % 128 != 0, F % 64 != 0 or g not in {64, 128}: kernel_path AUTO must still be right
    cross, err = small_layer_case(B, d=d, F=F, E=3, k=2, g=g, bits=(2, 4, 8), T=9)
    assert cross < TOL and err < TOL, (cross, err)
    cfg = B.Config(d, F, 3, 2, g, (2, 4, 8), kernel_path=2)
    x = torch.zeros((1, d), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.D2MoEError) as e:
        B.moe_forward(cfg, x, [x] * 9, logits=torch.zeros((1, 3), device="cuda"),
                      forced_bit_idx=torch.zeros((1, 2), dtype=torch.int8, device="cuda"))
    assert e.value.code == 4


@pytest.mark.gpu
@pytest.mark.parametrize("which", [0, 1])
def test_a_wait_that_nothing_satisfies_expires_and_leaves_the_device_usable(B, which):
    # the bounded waits of the expert kernels: after one second the block raises the timeout bit and returns
    import time
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    t0 = time.time()
    B.selftest_wait_expiry(which, status)
    torch.cuda.synchronize()
    dt = time.time() - t0
    assert int(status.item()) & 0x2, status
    assert 0.9 < dt < 5.0, dt          # one expiry, not two: the second wait sees the abort flag
    # the context is intact: a normal layer call still passes
    cross, err = small_layer_case(B, d=128, F=128, E=2, k=1, g=64, bits=(2, 4, 8), T=4)
    assert cross < TOL and err < TOL, (cross, err)


# ------------------------------------------------------------------ numeric range of the two expert kernels
def test_decode_kernel_outliers_of_1e3_and_1e4(B):
    # One element 10^3 / 10^4 times the rest of its token.  The decode kernel quantises a row to 15 bits against
    # its largest element; the noise this adds to an output is at most sqrt(n) / (16191 sqrt(12)) of the
    # output's rms (1.1e-3 at n = 4096, 2.1e-3 at n = 14336), because the outlier that sets the step also
    # carries the row's norm.  Both metrics must hold for every token.
    T = 8
    scales = [1.0] * T
    for outlier in [(1, 5, 1.0e3), (2, 700, 1.0e4), (3, 1023, -3.0e4)]:
        cross, err = small_layer_case(B, d=1024, F=1024, E=2, k=2, g=128, bits=(2, 3, 4, 8), T=T, token_scales=scales,
                                      outlier=outlier)
        assert err < TOL and cross < TOL, (outlier, cross, err)


def test_grouped_gemm_per_token_activation_scaling(B):
    # the grouped dequant-GEMM runs on fp16 tiles: every token row is scaled by a power of two of its own, so
    # tokens of magnitude 1e5 (beyond fp16), 1e-6 (below fp16's subnormals), an outlier of 1e4 and an all-zero
    # token in one prefill-sized batch all come out within tolerance, with no flag
    T = 400
    scales = [1.0] * T
    scales[3], scales[10], scales[50], scales[77], scales[200], scales[399] = 1.0e5, 1.0e-6, 0.0, 3.0e4, 2.0 ** -12, 7.0e8
    cross, err = small_layer_case(B, d=256, F=256, E=2, k=1, g=128, bits=(2, 3, 4, 8), T=T, probs=[0.1, 0.2, 0.4, 0.3],
                                  token_scales=scales, outlier=(5, 17, 1.0e4))
    assert err < TOL and cross < TOL, (cross, err)


def test_grouped_gemm_flags_nonfinite_activations(B):
    # a NaN / an infinity in a token at prefill size: flagged, that token's output is zero, the others are untouched
    d, F, E, k, g, bits, T = 256, 256, 2, 1, 128, (2, 4, 8), 300
    cfg = B.Config(d, F, E, k, g, bits)
    blobs = [B.pack_mwq(cfg, synth.normal(32, 100 + i, (F, d) if i % 3 < 2 else (d, F), 0.02, "cuda"))
             for i in range(3 * E)]
    x = synth.bf16_exact(synth.normal(32, 1, (T, d), 1.0, "cuda"))
    logits = synth.normal(32, 5, (T, E), 1.0, "cuda")
    fb = synth.categorical(32, 4, (T, k), [0.3, 0.3, 0.4], "cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    y_clean = B.moe_forward(cfg, x, blobs, logits=logits, forced_bit_idx=fb, device_status=st).clone()
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    x_bad = x.clone()
    x_bad[7, 5] = float("nan")
    x_bad[150, 9] = float("-inf")
    y_bad = B.moe_forward(cfg, x_bad, blobs, logits=logits, forced_bit_idx=fb, device_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) & B.DEV_NONFINITE
    keep = [t for t in range(T) if t not in (7, 150)]
    assert torch.equal(y_bad[keep], y_clean[keep])
    assert float(y_bad[[7, 150]].float().abs().max().item()) == 0.0


@pytest.mark.parametrize("T", [12, 300])
def test_bad_index_in_supplied_routing_is_flagged_and_skipped(B, T):
    # caller-supplied routing (`pre`) with one expert index and one width index out of range, on the tensor-core
    # kernels at decode size and at prefill size: the call is flagged and the two assignments contribute
    # nothing, exactly as if their gate weights were zero
    d, F, E, k, g, bits = 256, 256, 2, 2, 128, (2, 4, 8)
    cfg = B.Config(d, F, E, k, g, bits, kernel_path=2)
    blobs = [B.pack_mwq(cfg, synth.normal(33, 100 + i, (F, d) if i % 3 < 2 else (d, F), 0.02, "cuda"))
             for i in range(3 * E)]
    x = synth.bf16_exact(synth.normal(33, 1, (T, d), 1.0, "cuda"))
    logits = synth.normal(33, 5, (T, E), 1.0, "cuda")
    fb = synth.categorical(33, 4, (T, k), [0.3, 0.3, 0.4], "cuda")
    pre = B.route(cfg, x, logits=logits, forced_bit_idx=fb)
    torch.cuda.synchronize()
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    # reference: the same routing with the two assignments' weights set to zero
    ref = B.route(cfg, x, logits=logits, forced_bit_idx=fb)
    ref.topk_w[2, 1] = 0.0
    ref.topk_w[T - 1, 0] = 0.0
    y_ref = B.moe_forward(cfg, x, blobs, pre=ref, device_status=st).clone()
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    pre.topk_idx[2, 1] = E + 5
    pre.bit_idx[T - 1, 0] = 9
    y = B.moe_forward(cfg, x, blobs, pre=pre, device_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) & B.DEV_BAD_INDEX
    assert torch.equal(y, y_ref)


# ------------------------------------------------------------------ free per-step residual scales (scale_mode 1)
@pytest.mark.parametrize("bits,g,rows,cols", [((2, 3, 4, 8), 128, 256, 512), ((2, 4, 8), 64, 130, 256), ((2, 8), 32, 64, 96),
                                              ((1, 2, 3, 4, 5, 6, 7, 8), 256, 64, 512), ((3, 5), 64, 100, 128), ((4, 8), 128, 192, 1408)])
def test_pack_free_scales_bit_exact(B, bits, g, rows, cols):
    # codes, base scale / offset and every per-step scale of Eq. 4 / Eq. 5 against the oracle, bit for bit
    mwq, _, _ = oracle_mods()
    cfg = B.Config(cols, cols, 2, 1, g, bits, scale_mode=1)
    W = synth.normal(12, 5, (rows, cols), 0.02, "cuda")
    blob = B.pack_mwq(cfg, W)
    q = mwq.quantize(np_f32(W), bits, g, scale_mode=1)
    for b in range(bits[0], bits[-1] + 1):
        codes, s1, lo = B.unpack_codes(cfg, blob, rows, cols, b)
        assert np.array_equal(codes.cpu().numpy(), mwq.slice_code(q, b)), f"width {b}"
    assert np.array_equal(np_f32(s1), q.s1) and np.array_equal(np_f32(lo), q.lo)
    assert np.array_equal(np_f32(B.unpack_scales(cfg, blob, rows, cols)), q.s_extra)


@pytest.mark.parametrize("case", [
    dict(d=256, F=384, E=4, k=2, g=128, bits=(2, 3, 4, 8), T=24),                      # decode-sized: grouped GEMM all the same
    dict(d=256, F=256, E=2, k=1, g=128, bits=(2, 3, 4, 8), T=400, probs=[0.1, 0.2, 0.4, 0.3]),
    dict(d=256, F=384, E=4, k=2, g=64, bits=(2, 4, 8), T=50, n_shared=1),
    dict(d=256, F=256, E=2, k=2, g=128, bits=(1, 2, 3, 4, 5, 6, 7, 8), T=300),
    dict(d=128, F=128, E=2, k=1, g=64, bits=(3, 5), T=7),
    dict(d=192, F=256, E=3, k=2, g=64, bits=(2, 8), T=9),                              # CUDA-core path only (d % 128 != 0)
])
def test_free_scales_layer_against_oracle(B, case):
    cross, err = small_layer_case(B, scale_mode=1, **case)
    assert cross < TOL and err < TOL, (cross, err)


# ------------------------------------------------------------------ calibration-aware MWQ (Eq. 5 with energies, Algorithm 1)
@pytest.mark.parametrize("bits,g,rows,cols", [((2, 3, 4, 8), 128, 200, 512), ((2, 4, 8), 64, 64, 256), ((3, 5), 32, 130, 128)])
def test_pack_calibrated_bit_exact(B, bits, g, rows, cols):
    """Codes, base scales and every per-step scale of the calibrated packing against the oracle, bit for bit: with the
    Cholesky factor of a correlated synthetic activation set (error propagated block by block), with per-column
    energies in the scale fit, with both, and with neither (= the calibration-free packing)."""
    mwq, _, _ = oracle_mods()
    cfg = B.Config(cols, cols, 2, 1, g, bits, scale_mode=1)
    W = synth.normal(13, 5, (rows, cols), 0.02, "cuda")
    X = synth.normal(13, 6, (cols, 384), 1.0, "cpu").double()
    X = X + 0.6 * torch.roll(X, 1, 0) + 0.2 * torch.roll(X, 5, 0)
    X = X * (0.5 + 2.0 * synth.normal(13, 7, (cols, 1), 1.0, "cpu").abs().double())
    H = 2.0 * X @ X.T / X.shape[1] + 1e-2 * torch.eye(cols, dtype=torch.float64)
    hc = torch.linalg.cholesky(torch.linalg.inv(H), upper=True).float().contiguous()
    energy = (X * X).mean(dim=1).float().contiguous()
    for use_hc, use_e in ((True, False), (False, True), (True, True), (False, False)):
        blob = B.pack_mwq_calibrated(cfg, W, hc.cuda() if use_hc else None, energy.cuda() if use_e else None)
        q = mwq.quantize_calibrated(np_f32(W), bits, g, hc.numpy() if use_hc else None, energy.numpy() if use_e else None)
        codes, s1, lo = B.unpack_codes(cfg, blob, rows, cols, bits[-1])
        assert np.array_equal(codes.cpu().numpy(), q.code), (use_hc, use_e)
        assert np.array_equal(np_f32(s1), q.s1) and np.array_equal(np_f32(lo), q.lo)
        assert np.array_equal(np_f32(B.unpack_scales(cfg, blob, rows, cols)), q.s_extra)
        if not use_hc and not use_e:
            assert torch.equal(blob[256:], B.pack_mwq(cfg, W)[256:])
