"""Shared helpers of the tests: build a seeded case, move it to the GPU, compare with tolerances."""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np

from oracle import fff_oracle as orc
from paper_2308_14711_b200 import workloads as wl

ORACLE_THREADS = min(8, os.cpu_count() or 1)

# tolerances of the output comparison: |err| <= abs_rel * (1 + |ref|), and relative L2 over the tensor
TOL = {"f32": dict(abs_rel=1e-5, l2=None), "bf16": dict(abs_rel=2e-2, l2=1e-2)}


@dataclass
class Case:
    cfg: wl.FFFConfig
    weights: Dict[str, np.ndarray]
    net: orc.Net
    x: np.ndarray           # float32 [B, D], exactly representable in cfg.dtype, margin-enforced
    redrawn: int


def make_case(cfg: wl.FFFConfig, seed: int = 0, margin: Optional[float] = wl.DEFAULT_MARGIN) -> Case:
    weights = wl.make_weights(cfg, seed)
    net = orc.Net.from_config(cfg, weights)
    src = wl.TokenSource(cfg, seed)
    redrawn = 0
    if margin is not None:
        redrawn = wl.enforce_margin(src, lambda rows: orc.path_margin(net, rows, threads=ORACLE_THREADS), margin)
    return Case(cfg, weights, net, src.x, redrawn)


def to_device(a: np.ndarray, dtype: str):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype == "bf16":
        back = t.to(torch.bfloat16)
        assert torch.equal(back.float(), t), "inputs must already be bf16-representable"
        t = back
    return t.cuda()


def make_layer(case: Case, path: str = "auto"):
    from paper_2308_14711_b200.binding import FFFLayer
    cfg = case.cfg
    dev = {k: to_device(v, cfg.dtype) for k, v in case.weights.items()}
    if cfg.depth == 0:
        dev["node_w"] = dev["node_b"] = None
    return FFFLayer(cfg.D, cfg.O, cfg.depth, cfg.leaf_width, cfg.activation, cfg.dtype, path=path, **dev)


def check_outputs(y_gpu, y_ref: np.ndarray, dtype: str, rows: Optional[np.ndarray] = None, scale: float = 1.0) -> dict:
    """Element-wise tolerance check of y (torch tensor on any device) against float64 reference rows.
    scale > 1 widens both bounds for results that went through that many layers."""
    got = y_gpu.detach().float().cpu().numpy().astype(np.float64)
    if rows is not None:
        got = got[rows]
    assert got.shape == y_ref.shape
    assert np.isfinite(got).all()
    tol = TOL[dtype]
    err = np.abs(got - y_ref)
    bound = scale * tol["abs_rel"] * (1.0 + np.abs(y_ref))
    worst = float((err / bound).max()) if err.size else 0.0
    assert worst <= 1.0, f"max |err| is {worst:.3f}x the allowed {scale * tol['abs_rel']}*(1+|ref|)"
    rel_l2 = float(np.linalg.norm(got - y_ref) / max(np.linalg.norm(y_ref), 1e-300)) if err.size else 0.0
    if tol["l2"] is not None:
        assert rel_l2 <= scale * tol["l2"], f"relative L2 error {rel_l2:.3e} > {scale * tol['l2']}"
    return {"worst_over_bound": worst, "rel_l2": rel_l2}
