"""The seeded generators (no method arithmetic): determinism, slice
independence, distribution parameters and workload tables."""
import json
import os

import torch

from paper_2309_17224_b200 import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_same_seed_same_bits_and_chunking_does_not_matter():
    a = I.normal_bf16(300, 257, 0.02, I.BASE_SEED, 1234)
    b = I.normal_bf16(300, 257, 0.02, I.BASE_SEED, 1234, chunk_rows=7)
    c = I.normal_bf16(300, 257, 0.02, I.BASE_SEED + 1, 1234)
    d = I.normal_bf16(300, 257, 0.02, I.BASE_SEED, 1235)
    assert torch.equal(a, b)
    assert not torch.equal(a, c) and not torch.equal(a, d)
    # a leading slice is the same stream (element i depends on i only)
    assert torch.equal(I.normal_bf16(10, 257, 0.02, I.BASE_SEED, 1234), a[:10])


def test_distribution_and_outlier_columns():
    x = I.normal_bf16(4096, 1024, 1.0, 7, 1, outlier_frac=0.01, outlier_scale=50.0).float()
    mask = I.outlier_columns(1024, 0.01, 7, 1)
    assert 3 <= int(mask.sum()) <= 25
    assert abs(float(x[:, ~mask].std()) - 1.0) < 0.01 and abs(float(x[:, ~mask].mean())) < 0.01
    assert abs(float(x[:, mask].std()) - 50.0) < 2.5
    g = I.normal_bf16(512, 512, 1e-4, 7, 2, log2_scale=-6.0).float()
    assert abs(float(g.std()) / (1e-4 * 2.0 ** -6) - 1.0) < 0.02


def test_per_step_gradient_magnitude_is_log_uniform_in_range():
    wl = I.WORKLOADS["c2_gpt"]
    us = [I.uniform_scalar(I.BASE_SEED, I.tensor_id(2, 0, I.G_ID), s, *wl.g_log2_range) for s in range(200)]
    assert min(us) >= -12.0 and max(us) < -4.0 and len({round(u, 3) for u in us}) > 190
    assert -9.0 < sum(us) / len(us) < -7.0


def test_workloads_match_the_configs_they_stand_for():
    cfg = json.load(open(os.path.join(ROOT, "BASELINE.json")))["configs"]
    assert len(cfg) == 5
    c3 = I.WORKLOADS["c3_llama7b"]
    assert c3.tokens == 8192 and [(l.K, l.N) for l in c3.layers] == [(4096, 12288), (4096, 4096), (4096, 22016), (11008, 4096)]
    assert abs(c3.flops() - 9947e9) < 1e9           # forward + backward of the block
    c2 = I.WORKLOADS["c2_gpt"]
    assert abs(c2.flops() - 1237e9) < 1e9
    c4 = I.WORKLOADS["c4_llama70b_ptq"]
    assert not c4.backward and sum(l.K * l.N for l in c4.layers) == 855638016
    assert abs(c4.flops(2048) - 3505e9) < 1e9
    t = I.layer_tensors(I.WORKLOADS["c1_single"], 0)
    assert t["x"].shape == (256, 768) and t["w"].shape == (768, 768) and t["g"].shape == (256, 768)
    assert all(v.dtype == torch.bfloat16 for v in t.values())
