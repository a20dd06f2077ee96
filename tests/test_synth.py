"""The seeded input generators: determinism, slice-consistency, distribution sanity."""
import numpy as np
import torch

from paper_2504_15299_b200 import synth


def test_normal_is_deterministic_and_row_sliceable():
    a = synth.normal(3, 7, (50, 40), 0.02)
    b = synth.normal(3, 7, (50, 40), 0.02)
    assert torch.equal(a, b)
    rows = torch.tensor([49, 0, 17])
    c = synth.normal(3, 7, (50, 40), 0.02, rows=rows)
    assert torch.equal(c, a[rows])
    assert not torch.equal(a, synth.normal(4, 7, (50, 40), 0.02))
    assert not torch.equal(a, synth.normal(3, 8, (50, 40), 0.02))


def test_normal_moments():
    z = synth.normal(0, 1, (400, 1000), 1.0).double()
    assert abs(z.mean().item()) < 5e-3
    assert abs(z.std().item() - 1.0) < 5e-3
    assert abs((z ** 4).mean().item() - 3.0) < 0.05          # kurtosis of a normal
    assert z.abs().max().item() <= 4.5


def test_mixer_matches_python_reference():
    idx = torch.tensor([0, 1, 2, 12345678901], dtype=torch.int64)
    got = synth.random_bits(5, 9, idx).tolist()
    key = synth.stream_key(5, 9)
    for i, g in zip(idx.tolist(), got):
        ref = synth._mix64_py((i * 0x9E3779B97F4A7C15 + key) & ((1 << 64) - 1))
        assert (g & ((1 << 64) - 1)) == ref


def test_categorical_frequencies():
    c = synth.categorical(1, 4, (20000, 2), (0.1, 0.2, 0.4, 0.3)).long()
    freq = torch.bincount(c.reshape(-1), minlength=4).double() / c.numel()
    assert torch.allclose(freq, torch.tensor([0.1, 0.2, 0.4, 0.3], dtype=torch.float64), atol=0.01)


def test_workload_tensors():
    wl = synth.WORKLOADS["tiny"]
    x = synth.tokens_bf16(wl, 16)
    assert x.dtype == torch.bfloat16 and x.shape == (16, 256)
    W = synth.expert_matrix(wl, 1, 2)
    assert W.shape == (256, 512) and abs(W.std().item() - 0.02) < 1e-3
    assert synth.forced_bit_idx(wl, 16).shape == (16, 2)
    lg = synth.zipf_logits(synth.WORKLOADS["mixtral_prefill"], 64)
    assert lg.shape == (64, 8) and lg.dtype == torch.float32
