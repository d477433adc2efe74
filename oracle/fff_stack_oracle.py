"""CPU oracle for a stack of FFF blocks -- TEST INFRASTRUCTURE ONLY (see fff_oracle.c).

Section "Fast feedforward layers as building blocks" uses FFF layers in place of the feedforward layers of
a transformer: every such layer sits behind a layer normalisation and inside a residual connection.  With
the attention layers left out (they are not part of the FFF forward pass) a stack of K such blocks maps a
token x_0 to x_K by

    z_k     = LayerNorm_k(x_k)           = (x_k - mean(x_k)) / sqrt(var(x_k) + eps) * gamma_k + beta_k
    x_{k+1} = x_k + FFF_k(z_k)           (FORWARD_I of Algorithm 1 for layer k)

per token (mean and population variance over the D features).  Without normalisation z_k = x_k, without
residual x_{k+1} = FFF_k(z_k).

Everything is float64.  For a bf16 stack the tensors that the computation STORES between kernels are
values of that type, so z_k and x_{k+1} are rounded to bf16 (round to nearest even) where they are
produced; the arithmetic in between stays float64.  Tokens are independent of one another through the
whole stack.

Pinned by: torch.nn.functional.layer_norm (library routine), torch's bf16 conversion, a stack of one plain
block being FORWARD_I itself, and blocks with zero leaf parameters being the identity.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np

from oracle import fff_oracle as orc
from paper_2308_14711_b200 import workloads as wl      # storage rounding of the input generator


def layer_norm(x: np.ndarray, gamma: Optional[np.ndarray], beta: Optional[np.ndarray], eps: float) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    mean = x.mean(axis=1, keepdims=True)
    var = ((x - mean) ** 2).mean(axis=1, keepdims=True)
    z = (x - mean) / np.sqrt(var + eps)
    if gamma is not None:
        z = z * np.asarray(gamma, dtype=np.float64)
    if beta is not None:
        z = z + np.asarray(beta, dtype=np.float64)
    return z


def store(a: np.ndarray, dtype: str) -> np.ndarray:
    """The value a tensor of the stack's storage type holds after `a` has been written to it."""
    if dtype == "bf16":
        return wl.round_to_bf16(np.asarray(a, dtype=np.float64).astype(np.float32)).astype(np.float64)
    if dtype == "f32":
        return np.asarray(a, dtype=np.float64).astype(np.float32).astype(np.float64)
    raise ValueError(dtype)


def stack_forward(nets: Sequence[orc.Net], x, dtype: str, norms: Optional[Sequence[Optional[Tuple]]] = None,
                  eps: float = 1e-5, residual: bool = True, threads: int = 1):
    """Returns (x_K float64 [B, D], list of leaf_idx per block, smallest |routing logit| per token over all blocks).

    norms[k] is None (no normalisation in block k) or (gamma_k, beta_k), either of which may be None."""
    cur = np.asarray(x, dtype=np.float64)
    leaves: List[np.ndarray] = []
    margin = np.full(cur.shape[0], np.inf)
    for k, net in enumerate(nets):
        z = cur
        if norms is not None and norms[k] is not None:
            z = store(layer_norm(cur, norms[k][0], norms[k][1], eps), dtype)
        leaf, mn, _ = orc.descend(net, z, threads=threads)
        margin = np.minimum(margin, mn)
        y, leaf2 = orc.forward_i(net, z, threads=threads)
        assert np.array_equal(leaf, leaf2)
        leaves.append(leaf)
        cur = store(cur + y if residual else y, dtype)
    return cur, leaves, margin
