"""GPU parity at the full size of the five evaluated configurations, in the launch configuration the
benchmark times (default path, reserved workspace).

leaf_idx, the bucketing and y are compared for every token: the oracle evaluates the whole batch.
"""
import numpy as np
import pytest
import torch

from oracle import fff_oracle as orc
from paper_2308_14711_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", wl.CONFIG_ORDER)
def test_full_config(name):
    cfg = wl.CONFIGS[name]
    case = util.make_case(cfg, seed=0)
    leaf_ref, margin, _ = orc.descend(case.net, case.x, threads=util.ORACLE_THREADS)
    assert margin.min() >= wl.DEFAULT_MARGIN
    off_ref, perm_ref = orc.bucket(leaf_ref, cfg.n_leaves)

    layer = util.make_layer(case)
    layer.reserve(cfg.B)
    x = util.to_device(case.x, cfg.dtype)
    y, leaf = layer.forward_infer(x)
    torch.cuda.synchronize()
    assert layer.last_status() == 0
    np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
    off, perm = layer.last_bucketing(cfg.B)
    np.testing.assert_array_equal(off.cpu().numpy(), off_ref)
    np.testing.assert_array_equal(perm.cpu().numpy(), perm_ref)

    y_ref, leaf_all = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    np.testing.assert_array_equal(leaf_all, leaf_ref)
    util.check_outputs(y, y_ref, cfg.dtype)
    layer.close()


def test_large_batch_many_tiles_per_sm():
    """Half a million tokens of a small layer: many rounds of tiles per SM in every kernel, the first stage on
    CTA pairs with 255 nodes, more count rows than the ranked bucketing takes (it falls back to the grid-wide
    kernel), and an odd batch size."""
    cfg = wl.FFFConfig("bf16_large_batch", 128, 64, 8, 8, "gelu", "bf16", 500001, "normal")
    case = util.make_case(cfg, seed=5)
    leaf_ref, margin, _ = orc.descend(case.net, case.x, threads=util.ORACLE_THREADS)
    off_ref, perm_ref = orc.bucket(leaf_ref, cfg.n_leaves)
    layer = util.make_layer(case)
    x = util.to_device(case.x, cfg.dtype)
    for _ in range(2):
        y, leaf = layer.forward_infer(x)
        torch.cuda.synchronize()
        assert layer.last_status() == 0
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
        off, perm = layer.last_bucketing(cfg.B)
        np.testing.assert_array_equal(off.cpu().numpy(), off_ref)
        np.testing.assert_array_equal(perm.cpu().numpy(), perm_ref)
    y_ref, _ = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    util.check_outputs(y, y_ref, cfg.dtype)
    layer.close()
