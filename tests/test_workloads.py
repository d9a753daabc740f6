"""The seeded input generator: host and device implementations agree bit for bit, slices regenerate
independently, and the value distributions follow the stated recipe."""

import numpy as np
import pytest

from paper_2609_36222_b200 import workloads as wl


def test_numpy_and_torch_streams_are_bit_identical():
    torch = pytest.importorskip("torch")
    key = wl.stream_key(0, "qwen3", 3, "w_gate")
    a = wl.mix64_np(key, 12345, 4096)
    b = wl.mix64_torch(key, 12345, 4096, "cpu").numpy().view(np.uint64)
    np.testing.assert_array_equal(a, b)
    h = wl.normal_bf16_bits(key, 777, 100000, 0.02)
    d = wl.normal_bf16_device(key, 777, 100000, 0.02, "cpu")
    np.testing.assert_array_equal(h, d.view(torch.int16).numpy().view(np.uint16))


def test_bf16_packing_matches_torch_rounding():
    torch = pytest.importorskip("torch")
    x = (np.random.default_rng(0).standard_normal(50000) * 3).astype(np.float32)
    x[:4] = [1.00390625, 1.01171875, -0.0, 65504.0]      # ties-to-even cases
    bits = wl.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16)
    np.testing.assert_array_equal(bits, ref.view(torch.int16).numpy().view(np.uint16))
    np.testing.assert_array_equal(wl.bf16_bits_to_f32(bits), ref.float().numpy())


def test_slices_regenerate_independently():
    cfg = wl.CONFIGS["tiny"]
    full = wl.expert_weights_host_all(cfg)
    for u in (0, 5, 15):
        one = wl.expert_weights_host(cfg, u)
        for k in one:
            np.testing.assert_array_equal(one[k], full[k][u])
    assert full["w_gate"].shape == (16, 128, 256) and full["w_down"].shape == (16, 256, 128)
    other = wl.expert_weights_host(cfg, 0, layer=1)
    assert (other["w_gate"] != full["w_gate"][0]).mean() > 0.9


def test_value_distributions():
    cfg = wl.CONFIGS["tiny"]
    w = wl.bf16_bits_to_f64(wl.expert_weights_host_all(cfg)["w_up"]).ravel()
    assert abs(w.mean()) < 2e-4 and w.std() == pytest.approx(0.02, rel=0.01)
    assert np.abs(w).max() < 0.02 * 4.6
    assert abs(np.mean(np.abs(w) < 0.02) - 0.6827) < 0.005
    z = wl.bf16_bits_to_f64(wl.hidden_bits(wl.CONFIGS["qwen3"]))
    assert z.shape == (64, 2048)
    np.testing.assert_allclose(np.sqrt((z * z).mean(axis=1)), 1.0, rtol=2e-3)
    b = wl.router_bias(wl.CONFIGS["qwen3"])
    p = np.exp(b.astype(np.float64))
    p /= p.sum()
    ranks = np.arange(1, 129) ** -1.1
    np.testing.assert_allclose(np.sort(p)[::-1], ranks / ranks.sum(), rtol=1e-5)
    assert b.max() == 0.0 and len(set(b.tolist())) == 128


def test_configs_match_the_stated_shapes():
    c = wl.CONFIGS
    assert [c[n].name for n in wl.CONFIG_ORDER] == list(wl.CONFIG_ORDER)
    assert (c["qwen3"].d, c["qwen3"].E, c["qwen3"].K, c["qwen3"].I, c["qwen3"].T) == (2048, 128, 8, 768, 64)
    assert c["qwen3"].expert_bytes == 9437184
    assert c["mixtral"].expert_bytes == 352321536
    assert c["qwen3_stack"].layers == 48
