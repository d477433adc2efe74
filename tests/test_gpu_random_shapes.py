"""GPU parity on seeded random layer shapes: dimensions on and off the kernels' granules, depths 0-12,
hidden widths 1-64, batches from one token to several tile rounds per SM, all three input kinds.
Every case runs twice on the same handle (second call: warm workspace, rearmed scheduler words)."""
import numpy as np
import pytest
import torch

from oracle import fff_oracle as orc
from paper_2308_14711_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def random_cfgs(seed: int, n: int):
    rng = np.random.default_rng(seed)
    out = []
    for it in range(n):
        D = int(rng.choice([64, 128, 192, 256, 384, 512, 768, 1024]))
        O = int(rng.choice([16, 24, 48, 64, 80, 128, 208, 256, 520, 768, 1024]))
        depth = int(rng.integers(0, 13))
        l = int(rng.choice([1, 4, 8, 12, 16, 20, 32, 40, 64]))
        B = int(rng.choice([1, 37, 128, 129, 1000, 4097, 20000, 33333]))
        if (1 << depth) * l * (D + O) * 2 > 300e6:
            depth = min(depth, 8)
        kind = str(rng.choice(["normal", "layernorm", "clusters"]))
        act = str(rng.choice(["relu", "gelu"]))
        out.append(wl.FFFConfig(f"rand{seed}_{it}", D, O, depth, l, act, "bf16", B, kind,
                                node_bias_std=float(rng.choice([0.0, 0.3]))))
    return out


@pytest.mark.parametrize("cfg", random_cfgs(7, 24), ids=lambda c: f"{c.name}-D{c.D}-O{c.O}-d{c.depth}-l{c.leaf_width}-B{c.B}")
def test_random_shape(cfg):
    case = util.make_case(cfg, seed=11)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
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
        util.check_outputs(y, y_ref, cfg.dtype)
    layer.close()
