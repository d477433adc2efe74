"""GPU parity of layers whose leaf weights are stored as 8-bit floats (fff_create_w8) against the float64 oracle.

The generator encodes the leaf weights (e4m3 codes, one scale per leaf) and hands the oracle the exact values the
codes and scales stand for; the library gets the codes and scales.  Leaf indices bit-exact, outputs within the bf16
tolerance."""
import numpy as np
import pytest
import torch

from oracle import fff_oracle as orc
from paper_2308_14711_b200 import workloads as wl
from paper_2308_14711_b200.binding import FFFLayer, FFFError
from tests import util

pytestmark = pytest.mark.gpu

C = wl.FFFConfig
CASES = [
    C("w8_l32", 256, 128, 6, 32, "gelu", "bf16", 3001, "normal"),          # thin buckets: stacked short tiles
    C("w8_l12", 768, 768, 4, 12, "gelu", "bf16", 1500, "layernorm"),       # l below the padded width, six output pieces
    C("w8_l64", 128, 272, 3, 64, "relu", "bf16", 2000, "normal"),          # full width, O ends in a 16-column piece
    C("w8_skew", 128, 256, 7, 16, "silu", "bf16", 4099, "clusters"),       # a few large buckets, many empty leaves
    C("w8_d10", 128, 64, 10, 16, "gelu", "bf16", 20000, "clusters"),       # two descent stages in front
]


def make(cfg, seed):
    w = wl.make_weights(cfg, seed)
    c1, s1, v1 = wl.quantize_e4m3(w["w1"])
    c2, s2, v2 = wl.quantize_e4m3(w["w2"])
    net = orc.Net(cfg.D, cfg.O, cfg.depth, cfg.leaf_width, cfg.activation, w["node_w"], w["node_b"], v1, w["b1"], v2, w["b2"])
    src = wl.TokenSource(cfg, seed)
    wl.enforce_margin(src, lambda rows: orc.path_margin(net, rows, threads=util.ORACLE_THREADS))
    dev = {k: util.to_device(w[k], "bf16") for k in ("node_w", "node_b", "b1", "b2")}
    layer = FFFLayer(cfg.D, cfg.O, cfg.depth, cfg.leaf_width, cfg.activation, "bf16", dev["node_w"], dev["node_b"],
                     torch.from_numpy(c1).cuda(), dev["b1"], torch.from_numpy(c2).cuda(), dev["b2"],
                     w1_scale=torch.from_numpy(s1).cuda(), w2_scale=torch.from_numpy(s2).cuda())
    return net, src.x, layer


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
def test_w8_forward_matches_the_oracle(cfg):
    net, x_host, layer = make(cfg, seed=2)
    y_ref, leaf_ref = orc.forward_i(net, x_host, threads=util.ORACLE_THREADS)
    x = util.to_device(x_host, "bf16")
    y_first = None
    for _ in range(2):
        y, leaf = layer.forward_infer(x)
        torch.cuda.synchronize()
        assert layer.last_status() == 0
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
        util.check_outputs(y, y_ref, "bf16")
        off, perm = layer.last_bucketing(cfg.B)
        off_ref, perm_ref = orc.bucket(leaf_ref, cfg.n_leaves)
        np.testing.assert_array_equal(off.cpu().numpy(), off_ref)
        np.testing.assert_array_equal(perm.cpu().numpy(), perm_ref)
        assert y_first is None or torch.equal(y, y_first)
        y_first = y.clone()
    # the stage entry points on the same handle
    leaf2 = layer.tree_descent(x)
    off, perm = layer.leaf_bucketing(leaf2)
    y2 = layer.grouped_leaf_ff(x, leaf2, off, perm)
    util.check_outputs(y2, y_ref, "bf16")
    layer.close()


def test_w8_is_refused_where_the_tcgen05_leaf_kernel_cannot_run():
    cfg = C("w8_bad", 192, 64, 2, 8, "relu", "bf16", 4, "normal")           # D no multiple of 128
    w = wl.make_weights(cfg, 0)
    c1, s1, _ = wl.quantize_e4m3(w["w1"])
    c2, s2, _ = wl.quantize_e4m3(w["w2"])
    dev = {k: util.to_device(w[k], "bf16") for k in ("node_w", "node_b", "b1", "b2")}
    with pytest.raises(FFFError) as e:
        FFFLayer(cfg.D, cfg.O, cfg.depth, cfg.leaf_width, "relu", "bf16", dev["node_w"], dev["node_b"], torch.from_numpy(c1).cuda(),
                 dev["b1"], torch.from_numpy(c2).cuda(), dev["b2"], w1_scale=torch.from_numpy(s1).cuda(),
                 w2_scale=torch.from_numpy(s2).cuda())
    assert e.value.status == 2
