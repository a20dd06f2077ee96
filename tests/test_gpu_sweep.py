"""Batch-size sweep on small layers: the tensor-core path (which picks the decode kernel, in either of its two
instantiations, or the grouped GEMM from the load) against the plain CUDA-core path of the same library, every call
repeated and compared bit for bit.  The oracle is not involved: this test looks for size-dependent slips (unit
boundaries, padded width classes, crowded experts, the switch between kernels), the parity tests hold the values."""
import pytest
import torch

from paper_2504_15299_b200 import synth

pytestmark = pytest.mark.gpu

CASES = [(256, 384, 4, 2, 128, (2, 3, 4, 8), 0), (256, 256, 8, 2, 64, (2, 4, 8), 1),
         (512, 256, 16, 4, 128, (5, 6, 7, 8), 0), (256, 256, 6, 3, 128, (1, 2, 3, 4, 5, 6, 7, 8), 2)]
TOKENS = list(range(1, 40)) + [47, 48, 49, 63, 64, 65, 96, 127, 128, 129, 200, 333]


@pytest.fixture(scope="module")
def B():
    from paper_2504_15299_b200 import binding, build
    build.build_library()
    binding.lib()
    return binding


@pytest.mark.parametrize("d,F,E,k,g,bits,n_shared", CASES)
def test_every_batch_size_agrees_with_the_cuda_core_path_and_with_itself(B, d, F, E, k, g, bits, n_shared):
    cfg_tc = B.Config(d, F, E, k, g, bits, n_shared=n_shared, kernel_path=0)
    cfg_cc = B.Config(d, F, E, k, g, bits, n_shared=n_shared, kernel_path=1)
    blobs = []
    for e in range(E + n_shared):
        for m in range(3):
            shape = (F, d) if m < 2 else (d, F)
            blobs.append(B.pack_mwq(cfg_tc, synth.normal(7, 100 + 3 * e + m, shape, 0.02, "cuda")))
    K = len(bits)
    for T in TOKENS:
        x = synth.bf16_exact(synth.normal(7, 1000 + T, (T, d), 1.0, "cuda"))
        logits = synth.normal(7, 2000 + T, (T, E), 1.0, "cuda")
        if T % 5 == 0:
            logits[:, 0] += 50.0                     # every token picks expert 0 first: a crowded expert
        fb = synth.categorical(7, 3000 + T, (T, k), [1.0 / K] * K, "cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        y1 = B.moe_forward(cfg_tc, x, blobs, logits=logits, forced_bit_idx=fb, device_status=st)
        y1b = B.moe_forward(cfg_tc, x, blobs, logits=logits, forced_bit_idx=fb, device_status=st)
        y2 = B.moe_forward(cfg_cc, x, blobs, logits=logits, forced_bit_idx=fb, device_status=st).float()
        torch.cuda.synchronize()
        assert int(st.item()) == 0, (T, int(st.item()))
        assert torch.equal(y1.view(torch.int16), y1b.view(torch.int16)), ("rerun differs", T)
        err = float(((y1.float() - y2).abs().amax(dim=1) / y2.abs().amax(dim=1).clamp_min(1e-30)).max())
        assert err <= 1e-2, (T, err)
