"""The seeded input generator: determinism, chunk independence, distribution moments."""
import math

import torch

from paper_2501_00692_b200 import synth


def test_counter_based_and_chunk_independent():
    a = synth.normal(123, 0, 1000, "cpu")
    b = torch.cat([synth.normal(123, 0, 400, "cpu"), synth.normal(123, 400, 600, "cpu")])
    assert torch.equal(a, b)
    assert not torch.equal(a, synth.normal(124, 0, 1000, "cpu"))


def test_moments():
    n = 1 << 18
    z = synth.normal(5, 0, n, "cpu")
    assert abs(z.mean().item()) < 4 / math.sqrt(n)
    assert abs(z.var().item() - 1) < 0.02
    u = synth.uniform01(5, 0, n, "cpu")
    assert 0 < u.min().item() and u.max().item() < 1
    assert abs(u.mean().item() - 0.5) < 0.01


def test_workload_recipe():
    w = synth.WORKLOADS["C1"]
    th = synth.layer_params(w)
    assert th["W_delta"].shape == (64, 64) and th["A_log"].shape == (64, 16)
    assert -4 <= th["b_delta"].min().item() and th["b_delta"].max().item() <= -2
    assert 0 <= th["A_log"].min().item() and th["A_log"].max().item() <= math.log(16) + 1e-6
    assert abs(th["W_B"].double().std().item() - 1 / 8) < 0.01
    ths = synth.layer_params(w, slow_decay=True)
    assert ths["b_delta"].max().item() <= -7 and torch.equal(ths["W_B"], th["W_B"])
    x, dy = synth.activations(w)
    assert x.shape == (1, 512, 64) and x.dtype == torch.float32 and not torch.equal(x, dy)
    w3 = synth.custom_workload("t", 3, 1, 8, 16, io="bf16")
    assert synth.layer_params(w3)["W_C"].dtype == torch.bfloat16
    assert synth.layer_params(w3, layer=1)["W_C"].ne(synth.layer_params(w3)["W_C"]).any()
