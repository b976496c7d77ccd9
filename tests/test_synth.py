"""The seeded input generators: reproducible, chunk-independent, with the stated distributions."""
import math

import numpy as np
import torch

import synth


def test_hash_is_a_pure_function_of_the_counter():
    a = synth.hash_u32(1, 2, 3, 0, 1000)
    b = synth.hash_u32(1, 2, 3, 500, 100)
    assert torch.equal(a[500:600], b)
    assert not torch.equal(a, synth.hash_u32(1, 2, 4, 0, 1000))
    assert not torch.equal(a, synth.hash_u32(2, 2, 3, 0, 1000))
    assert int(a.min()) >= 0 and int(a.max()) < 2 ** 32
    big = synth.hash_u32(1, 2, 3, (1 << 33) + 5, 4)
    assert not torch.equal(big, synth.hash_u32(1, 2, 3, 5, 4))     # high counter bits matter


def test_normal_bf16_moments_and_reproducibility():
    x = synth.normal_bf16(5, 9, 400_000, 0.02)
    assert x.dtype == torch.bfloat16
    f = x.double()
    assert abs(f.mean().item()) < 2e-4
    assert abs(f.std().item() - 0.02) < 2e-4
    assert f.abs().max().item() <= 6 * 0.02 * 1.01
    assert torch.equal(x, synth.normal_bf16(5, 9, 400_000, 0.02))
    # kurtosis of a 12-term Irwin-Hall sum is 3 - 0.1
    k = ((f / f.std()) ** 4).mean().item()
    assert 2.8 < k < 3.0


def test_gumbel_noise_moments_and_finiteness():
    g = synth.gumbel_noise(1, 0, 1000, 1000).double()
    mean, var = synth.expected_gumbel_moments()
    assert torch.isfinite(g).all()
    assert abs(g.mean().item() - mean) < 5e-3
    assert abs(g.var().item() - var) < 2e-2
    assert not torch.equal(g, synth.gumbel_noise(1, 1, 1000, 1000).double())
    # extreme counters stay finite: u in [2^-25, 1 - 2^-25]
    lo = -math.log(-math.log(0.5 * 2 ** -24)); hi = -math.log(-math.log(1 - 0.5 * 2 ** -24))
    assert g.min().item() >= lo - 1e-6 and g.max().item() <= hi + 1e-6


def test_tokens_and_lengths_ranges():
    t = synth.token_ids(3, 0, 50_000, 4096)
    assert t.dtype == torch.int32 and int(t.min()) >= 0 and int(t.max()) < 4096
    counts = np.bincount(t.numpy(), minlength=4096)
    assert counts.min() > 0
    ls = synth.lengths(3, 0, 5000, 64, 128)
    assert min(ls) == 64 and max(ls) == 128


def test_weight_shapes_and_byte_counts():
    d = synth.shape("tiny")
    w = synth.make_weights(d)
    assert w["embed"].shape == (4096, 256) and w["lm_head"] is None
    assert w["wq"][1].shape == (256, 256) and w["wk"][0].shape == (128, 256)
    assert w["w_gate"][0].shape == (688, 256) and w["w_down"][0].shape == (256, 688)
    assert torch.all(w["ln1"][0] == 1)
    assert not torch.equal(w["wq"][0], w["wq"][1])
    q = synth.shape("qwen3_4b")
    assert synth.weight_bytes_per_step(q) == 8_044_544_000
    assert synth.kv_bytes_per_token(q) == 147_456
    assert synth.kv_bytes_per_token(synth.shape("llama31_8b")) == 131_072
    assert synth.kv_bytes_per_token(synth.shape("qwen25_7b")) == 57_344
