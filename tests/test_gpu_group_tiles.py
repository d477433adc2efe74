"""GPU parity of the leaf kernel's grouped tiles (tokens that share the node three levels above the leaves; the leaf
kernel walks the last three levels itself and evaluates the node's 8 leaves side by side) against the float64 oracle.

Leaf indices and the bucketing bit-exact, outputs within the bf16 tolerance, and the same results bit for bit as the
one-leaf-per-tile kernel gives for the leaf indices (outputs of the two may differ in the last bf16 digit: the
contraction over 8 x 16 hidden columns adds zeros in a different order)."""
import numpy as np
import pytest
import torch

from oracle import fff_oracle as orc
from paper_2308_14711_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu

C = wl.FFFConfig
CASES = [
    C("g_d9", 128, 64, 9, 12, "gelu", "bf16", 9000, "normal"),             # 64 nodes, ragged tiles, one 64-column piece
    C("g_d9_vit", 768, 768, 9, 12, "gelu", "bf16", 8300, "layernorm"),     # the ViT widths: twelve K-blocks, six pieces
    C("g_d9_min", 128, 128, 9, 9, "gelu_tanh", "bf16", 8192, "normal"),    # exactly 128 tokens per node on average
    C("g_d10", 256, 80, 10, 8, "relu", "bf16", 17000, "normal"),           # O ends in a 16-column piece
    C("g_d10_skew", 128, 272, 10, 15, "silu", "bf16", 20000, "clusters"),  # skewed routing: empty and thin nodes, 3 pieces
    C("g_d11", 128, 64, 11, 8, "gelu", "bf16", 40000, "normal"),           # 256 nodes: first stage of 8 levels on CTA pairs
    C("g_d11_wide", 1024, 1024, 11, 12, "gelu", "bf16", 65536, "normal"),  # full size: 512 full tiles, every row compared
]


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
def test_grouped_tiles_match_the_oracle(cfg):
    case = util.make_case(cfg, seed=5)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    off_ref, perm_ref = orc.bucket(leaf_ref, cfg.n_leaves)
    layer = util.make_layer(case)
    assert layer.capabilities() & 64                   # FFF_CAP_GROUP_TILES
    x = util.to_device(case.x, "bf16")
    y_first = None
    for _ in range(2):
        y, leaf = layer.forward_infer(x)
        torch.cuda.synchronize()
        assert layer.last_status() == 0
        assert layer.last_launch_count() == 2          # first descent stage + leaf kernel: the grouped path ran
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
        util.check_outputs(y, y_ref, "bf16")
        off, perm = layer.last_bucketing(cfg.B)
        np.testing.assert_array_equal(off.cpu().numpy(), off_ref)
        np.testing.assert_array_equal(perm.cpu().numpy(), perm_ref)
        assert y_first is None or torch.equal(y, y_first)
        y_first = y.clone()
    # without the caller's leaf_idx buffer the leaves still reach the workspace (bucketing on demand)
    y2, none = layer.forward_infer(x, want_leaf_idx=False)
    assert none is None and torch.equal(y2, y_first)
    off, perm = layer.last_bucketing(cfg.B)
    np.testing.assert_array_equal(perm.cpu().numpy(), perm_ref)
    # the one-leaf-per-tile kernel on the same handle
    layer.set_tuning("group_tiles", False)
    y3, leaf3 = layer.forward_infer(x)
    torch.cuda.synchronize()
    assert layer.last_launch_count() >= 3          # two descent stages and the leaf kernel
    np.testing.assert_array_equal(leaf3.cpu().numpy(), leaf_ref)
    util.check_outputs(y3, y_ref, "bf16")
    layer.close()


def test_too_few_tokens_per_node_keep_one_leaf_per_tile():
    """Below 128 tokens per node of the third level from the bottom the grouped path is not taken."""
    cfg = C("g_thin", 128, 64, 9, 12, "gelu", "bf16", 8000, "normal")       # 64 nodes x 128 = 8192 > 8000
    case = util.make_case(cfg, seed=6)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    layer = util.make_layer(case)
    y, leaf = layer.forward_infer(util.to_device(case.x, "bf16"))
    torch.cuda.synchronize()
    assert layer.last_launch_count() >= 3
    np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
    util.check_outputs(y, y_ref, "bf16")
    layer.set_tuning("group_tiles", False)
    y2, _ = layer.forward_infer(util.to_device(case.x, "bf16"))
    assert torch.equal(y, y2)
    layer.close()
