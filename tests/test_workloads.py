"""Host-side checks of the seeded workload generator (no GPU, no method arithmetic)."""
import numpy as np
import pytest
import torch

from oracle import fff_oracle as orc
from paper_2308_14711_b200 import workloads as wl


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    a = (rng.standard_normal(100000) * np.exp(rng.uniform(-20, 20, 100000))).astype(np.float32)
    a[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]      # ties: to even
    ref = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    got = wl.round_to_bf16(a)
    np.testing.assert_array_equal(got, ref)
    bits = wl.bf16_bits(got)
    np.testing.assert_array_equal(wl.bf16_bits_to_f32(bits), got)
    np.testing.assert_array_equal(torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).float().numpy(), got)


def test_five_configs_have_the_stated_shapes():
    c = wl.CONFIGS
    assert [(*(getattr(v, k) for k in ("D", "O", "depth", "leaf_width", "B")), v.dtype, v.activation)
            for v in c.values()] == [
        (784, 10, 3, 32, 2048, "f32", "relu"),
        (768, 768, 8, 12, 50432, "bf16", "gelu"),
        (1024, 1024, 11, 32, 65536, "bf16", "gelu"),
        (768, 768, 15, 1, 16384, "bf16", "gelu"),
        (1024, 1024, 11, 32, 65536, "bf16", "gelu"),
    ]
    assert c["vit_d8_l12_bf16"].n_leaves * 12 == 3072
    assert c["wide_d11_l32_bf16"].n_leaves * 32 == 65536


def test_generation_is_deterministic_and_prefix_stable():
    cfg = wl.CONFIGS["mnist_d3_l32_f32"]
    w0, w1 = wl.make_weights(cfg, 0), wl.make_weights(cfg, 0)
    for k in w0:
        np.testing.assert_array_equal(w0[k], w1[k])
    assert w0["w1"].shape == (8, 32, 784) and w0["w2"].shape == (8, 10, 32)
    assert not np.array_equal(wl.make_weights(cfg, 1)["w1"], w0["w1"])
    a = wl.TokenSource(cfg, 0).x
    b = wl.TokenSource(cfg, 0, B=100).x
    np.testing.assert_array_equal(a[:100], b)
    assert (w0["node_b"] == 0).all()


def test_value_distributions():
    cfg = wl.CONFIGS["vit_d8_l12_bf16"].with_batch(512)
    w = wl.make_weights(cfg, 0)
    assert abs(w["node_w"].std() * np.sqrt(768) - 1) < 0.02
    assert abs(w["w1"].std() * np.sqrt(768) - 1) < 0.02
    assert abs(w["w2"].std() * np.sqrt(12) - 1) < 0.02
    assert abs(w["b2"].std() / 0.1 - 1) < 0.05
    x = wl.TokenSource(cfg, 0).x
    assert np.abs(x.mean(axis=1)).max() < 5e-3 and np.abs(x.std(axis=1) - 1).max() < 5e-3
    # everything is bf16-representable
    for a in list(w.values()) + [x]:
        np.testing.assert_array_equal(wl.round_to_bf16(a), a)


def test_cluster_mixture_follows_zipf_weights():
    cfg = wl.CONFIGS["skew_d11_l32_bf16"].with_batch(20000)
    src = wl.TokenSource(cfg, 0)
    freq = np.bincount(src.cluster, minlength=16) / 20000
    np.testing.assert_allclose(freq, wl.zipf_weights(), atol=0.012)
    assert abs(wl.zipf_weights()[0] - 0.365) < 2e-3
    d = src.x - src.centres[src.cluster]
    assert abs(d.std() - 0.1) < 5e-3


def test_margin_resampling_with_the_oracle_margin():
    cfg = wl.FFFConfig("t", 32, 8, 6, 4, "gelu", "bf16", 4000, "clusters")
    w = wl.make_weights(cfg, 0)
    net = orc.Net.from_config(cfg, w)
    src = wl.TokenSource(cfg, 0)
    before = src.x.copy()
    cl = src.cluster.copy()
    m0 = orc.path_margin(net, before)
    n = wl.enforce_margin(src, lambda rows: orc.path_margin(net, rows))
    assert n == int((m0 < 1e-2).sum()) and n > 0
    assert orc.path_margin(net, src.x).min() >= 1e-2
    keep = m0 >= 1e-2
    np.testing.assert_array_equal(src.x[keep], before[keep])
    np.testing.assert_array_equal(src.cluster, cl)
    np.testing.assert_array_equal(wl.round_to_bf16(src.x), src.x)


def test_e4m3_codes_are_the_published_format_and_quantisation_is_nearest():
    """The 8-bit weight encoding of the generator: every code decodes to (-1)^s 2^(e-7) (1 + m/8), subnormals
    m/8 2^-6 (the published e4m3 format: 4 exponent bits with bias 7, 3 mantissa bits, no infinities, largest
    finite value 448); quantised values are the nearest representable ones and the per-leaf scale maps the largest
    magnitude of a leaf to 448."""
    table = wl.e4m3_decode_table()
    for code in range(256):
        s, e, m = code >> 7, (code >> 3) & 15, code & 7
        if e == 15 and m == 7:
            assert np.isnan(table[code])
            continue
        mag = (m / 8.0) * 2.0 ** -6 if e == 0 else 2.0 ** (e - 7) * (1.0 + m / 8.0)
        assert table[code] == (-mag if s else mag)
    assert np.nanmax(table) == 448.0
    rng = np.random.default_rng(0)
    w = (rng.standard_normal((5, 7, 33)) * rng.uniform(0.01, 3.0, (5, 1, 1))).astype(np.float32)
    w[3] = 0.0
    codes, scales, values = wl.quantize_e4m3(w)
    assert codes.dtype == np.uint8 and codes.shape == w.shape and scales.shape == (5,) and values.dtype == np.float64
    assert scales[3] == 1.0 and (values[3] == 0).all()
    finite = np.sort(table[np.isfinite(table)].astype(np.float64))
    for j in (0, 1, 2, 4):
        np.testing.assert_allclose(np.abs(values[j]).max(), np.abs(w[j]).max(), rtol=1e-6)
        target = w[j].astype(np.float64) / float(scales[j])
        got = values[j] / float(scales[j])
        # no representable value is closer to the target than the chosen one
        nearest = np.abs(finite[None, :] - target.reshape(-1, 1)).min(axis=1)
        np.testing.assert_allclose(np.abs(got - target).reshape(-1), nearest, rtol=0, atol=1e-6)
        np.testing.assert_array_equal(values[j], table[codes[j]].astype(np.float64) * float(scales[j]))
