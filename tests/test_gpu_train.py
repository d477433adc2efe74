"""GPU parity of FORWARD_T (the training-time forward pass: every leaf evaluated, outputs mixed by the node
choices) against the float64 oracle: outputs within the bf16 tolerance, mixture weights and node entropies to
float32 accuracy.  No routing decision is taken on this path, so the inputs need no margin."""
import numpy as np
import pytest
import torch

from oracle import fff_oracle as orc
from paper_2308_14711_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu

C = wl.FFFConfig
CASES = [
    C("train_d3_l8", 128, 64, 3, 8, "gelu", "bf16", 700, "normal", node_bias_std=0.3),
    C("train_d5_l12", 256, 272, 5, 12, "relu", "bf16", 1500, "layernorm"),          # O ends in a 16-column piece
    C("train_d2_l1", 64, 16, 2, 1, "silu", "bf16", 333, "normal", node_bias_std=0.5),
    C("train_d0", 128, 40, 0, 24, "gelu_tanh", "bf16", 200, "normal"),              # no nodes: one leaf with weight 1
    C("train_d8_l3", 192, 96, 8, 3, "gelu", "bf16", 450, "normal"),                 # 255 nodes, 768 hidden neurons + 256 mixture columns
]


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
def test_forward_train_matches_the_oracle(cfg):
    case = util.make_case(cfg, seed=3, margin=None)
    y_ref = orc.forward_t_rows(case.net, case.x, threads=util.ORACLE_THREADS)
    mix_ref = orc.mixture_weights(case.net, case.x, threads=util.ORACLE_THREADS)
    ent_ref = orc.node_entropy(case.net, case.x)
    layer = util.make_layer(case)
    x = util.to_device(case.x, "bf16")
    for _ in range(2):
        y, mix, ent = layer.forward_train(x)
        torch.cuda.synchronize()
        assert layer.last_status() == 0
        util.check_outputs(y, y_ref, "bf16")
        np.testing.assert_allclose(mix.cpu().numpy(), mix_ref, rtol=2e-4, atol=2e-6)
        np.testing.assert_allclose(mix.sum(dim=1).cpu().numpy(), 1.0, rtol=0, atol=1e-5)
        if cfg.depth > 0:
            np.testing.assert_allclose(ent.cpu().numpy(), ent_ref, rtol=1e-3, atol=1e-6)
    # outputs alone; and the hard forward on the same handle is untouched by the training workspace
    y_only, none_m, none_e = layer.forward_train(x, want_mixture=False, want_entropy=False)
    assert none_m is None and none_e is None and torch.equal(y_only, y)
    layer.close()


def test_forward_train_saturated_nodes_give_the_hard_forward():
    """Node weights scaled far into saturation: every choice is 0 or 1, the mixture is the indicator of the leaf the
    hard descent reaches, and FORWARD_T returns FORWARD_I's output (Section "Hardening")."""
    cfg = C("train_saturated", 128, 64, 4, 16, "gelu", "bf16", 900, "normal")
    case = util.make_case(cfg, seed=6)
    case.weights["node_w"] = wl.round_to_bf16(case.weights["node_w"] * np.float32(4096.0))
    case.net = orc.Net.from_config(cfg, case.weights)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    layer = util.make_layer(case)
    x = util.to_device(case.x, "bf16")
    y, mix, ent = layer.forward_train(x)
    y_hard, leaf = layer.forward_infer(x)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
    np.testing.assert_array_equal(mix.argmax(dim=1).cpu().numpy(), leaf_ref)
    assert float(mix.max(dim=1).values.min()) > 1.0 - 1e-6
    # (every node sees every token, also tokens that pass it by and may sit close to its boundary)
    assert float(ent.max()) < 1e-2
    np.testing.assert_allclose(ent.cpu().numpy(), orc.node_entropy(case.net, case.x), rtol=2e-2, atol=1e-6)
    util.check_outputs(y, y_ref, "bf16")
    util.check_outputs(y_hard, y_ref, "bf16")
    layer.close()


def test_forward_train_rejects_layers_it_cannot_run():
    from paper_2308_14711_b200.binding import FFFError
    cfg = C("train_f32", 64, 16, 2, 4, "relu", "f32", 10, "normal")
    layer = util.make_layer(util.make_case(cfg, seed=1, margin=None))
    with pytest.raises(FFFError) as e:
        layer.forward_train(util.to_device(np.zeros((10, 64), np.float32), "f32"))
    assert e.value.status == 2
    layer.close()
