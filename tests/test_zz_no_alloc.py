"""The workspace-free routing entry point (d2moe_route_static_scratch), for callers that may not
allocate device memory when they route a batch (frozen memory pools, plug-ins inside another
framework's step).  It must give exactly what d2moe_route gives, on back-to-back calls that share
its built-in scratch array.  This file sorts last on purpose: a run that stops at the first failure
has then already gone through every other test."""
import pytest
import torch

from paper_2504_15299_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2504_15299_b200 import binding, build
    build.build_library()
    binding.lib()
    return binding


def same_routing(a, b):
    assert torch.equal(a.topk_idx, b.topk_idx) and torch.equal(a.bit_idx, b.bit_idx)
    assert torch.equal(a.perm, b.perm) and torch.equal(a.inv_perm, b.inv_perm)
    assert torch.equal(a.group_off, b.group_off)
    assert torch.allclose(a.topk_w, b.topk_w, rtol=1e-5, atol=1e-7)
    assert int(a.device_status.item()) == 0 and int(b.device_status.item()) == 0


def test_static_scratch_routing_matches_workspace_routing_twice_in_a_row(B):
    # first call: the fine-grained layer (64 experts, top-6, 3 widths, 256 tokens)
    wl = synth.WORKLOADS["finegrained"]
    cfg = B.Config.from_workload(wl)
    x = synth.tokens_bf16(wl, 256, "cuda")
    gw = synth.gate_weight_bf16(wl, "cuda")
    fb = synth.forced_bit_idx(wl, 256, "cuda")
    ref1 = B.route(cfg, x, gate_w=gw, forced_bit_idx=fb)
    got1 = B.route_static_scratch(cfg, x, gate_w=gw, forced_bit_idx=fb)
    # second call right behind it, a different and smaller problem: whatever the first call left in
    # the shared scratch must not leak into it
    wl2 = synth.WORKLOADS["mixtral_stack"]
    cfg2 = B.Config.from_workload(wl2)
    x2 = synth.tokens_bf16(wl2, 16, "cuda")
    gw2 = synth.gate_weight_bf16(wl2, "cuda")
    bw2 = synth.bit_router_weight_bf16(wl2, "cuda")
    got2 = B.route_static_scratch(cfg2, x2, gate_w=gw2, bit_w=bw2)
    ref2 = B.route(cfg2, x2, gate_w=gw2, bit_w=bw2)
    torch.cuda.synchronize()
    same_routing(got1, ref1)
    same_routing(got2, ref2)
    # and the first problem again, reusing the output tensors (no allocation on either side)
    got3 = B.route_static_scratch(cfg, x, gate_w=gw, forced_bit_idx=fb, out=got1)
    torch.cuda.synchronize()
    same_routing(got3, ref1)


def test_static_scratch_refuses_what_does_not_fit(B):
    wl = synth.WORKLOADS["mixtral_prefill"]
    cfg = B.Config.from_workload(wl)
    T = B.STATIC_MAX_ASSIGNMENTS // cfg.top_k + 1
    x = torch.zeros((T, wl.d_model), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.D2MoEError) as err:
        B.route_static_scratch(cfg, x, logits=torch.zeros((T, 8), device="cuda"),
                               forced_bit_idx=torch.zeros((T, 2), dtype=torch.int8, device="cuda"))
    assert err.value.code == 5
