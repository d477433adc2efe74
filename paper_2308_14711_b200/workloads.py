"""Seeded synthetic workloads for FFF hard-routed inference.

This module only draws random numbers and lays them out: shapes, value
distributions and routing structure of the evaluated configurations.  It
contains none of the method's arithmetic (no tree descent, no leaf evaluation,
no bucketing) and imports neither the CPU oracle nor the CUDA binding, so both
can be fed from it.

The paper evaluates trained networks on image datasets (MNIST-shaped
784 -> 10 layers, BERT-base-shaped 768 -> 768 layers, ViT feedforward layers).
Neither the data nor the trained weights are available, so tensors of the same
shapes are drawn from fixed distributions instead:

  * a normal distribution written N(0, v) has *variance* v;
  * node weights ~ N(0, 1/D), node biases 0;
  * leaf W1 ~ N(0, 1/D), W2 ~ N(0, 1/l), leaf biases ~ N(0, 0.01);
  * tokens are iid N(0,1) rows ("normal"), per-token standardised rows
    ("layernorm": zero mean, unit population variance over D, no affine), or a
    16-component Gaussian mixture with Zipf(1.2) weights ("clusters":
    centres ~ N(0, I), within-cluster sigma 0.1);
  * for bf16 configurations every tensor is rounded to bf16 (round to nearest,
    ties to even) here, so that every consumer sees exactly the same values.

Every tensor has its own counter-based (Philox) stream keyed by
(seed, tensor id), so changing one shape does not shift another tensor.

Tokens whose routing would be decided by a near-zero node logit can be redrawn
(`enforce_margin`).  The margin itself is computed by a function the caller
passes in; this module only performs the redraw.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Callable, Dict, Optional

import numpy as np

# stream ids (second word of the Philox key)
_S_X, _S_NODE_W, _S_NODE_B, _S_W1, _S_B1, _S_W2, _S_B2, _S_CENTRES, _S_PICKS, _S_REDRAW = range(10)

N_CLUSTERS = 16
CLUSTER_SIGMA = 0.1
ZIPF_S = 1.2
LEAF_BIAS_STD = 0.1          # N(0, 0.01)
DEFAULT_MARGIN = 1e-2


@dataclass(frozen=True)
class FFFConfig:
    """Shape and input recipe of one FFF layer workload."""
    name: str
    D: int                    # dim_I
    O: int                    # dim_O
    depth: int                # d >= 0
    leaf_width: int           # l
    activation: str           # "relu" | "gelu" | "gelu_tanh" | "silu"
    dtype: str                # "f32" | "bf16"
    B: int                    # tokens per batch
    x_kind: str = "normal"    # "normal" | "layernorm" | "clusters"
    node_bias_std: float = 0.0

    @property
    def n_nodes(self) -> int:
        return (1 << self.depth) - 1

    @property
    def n_leaves(self) -> int:
        return 1 << self.depth

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def with_batch(self, B: int) -> "FFFConfig":
        return replace(self, B=B)


# The five evaluated configurations.
CONFIGS: Dict[str, FFFConfig] = {
    "mnist_d3_l32_f32": FFFConfig("mnist_d3_l32_f32", 784, 10, 3, 32, "relu", "f32", 2048, "normal"),
    "vit_d8_l12_bf16": FFFConfig("vit_d8_l12_bf16", 768, 768, 8, 12, "gelu", "bf16", 256 * 197, "layernorm"),
    "wide_d11_l32_bf16": FFFConfig("wide_d11_l32_bf16", 1024, 1024, 11, 32, "gelu", "bf16", 65536, "normal"),
    "deep_d15_l1_bf16": FFFConfig("deep_d15_l1_bf16", 768, 768, 15, 1, "gelu", "bf16", 16384, "normal"),
    "skew_d11_l32_bf16": FFFConfig("skew_d11_l32_bf16", 1024, 1024, 11, 32, "gelu", "bf16", 65536, "clusters"),
}
CONFIG_ORDER = list(CONFIGS)


def _rng(seed: int, stream: int, sub: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream) + (int(sub) << 16)]))


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    assert not np.any(u & np.uint32(0xFFFF)), "values are not bf16-representable"
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _store(cfg: FFFConfig, a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return round_to_bf16(a) if cfg.dtype == "bf16" else a


def _normal(seed: int, stream: int, shape, std: float, sub: int = 0) -> np.ndarray:
    g = _rng(seed, stream, sub).standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        g *= np.float32(std)
    return g


def make_weights(cfg: FFFConfig, seed: int = 0) -> Dict[str, np.ndarray]:
    """Node and leaf parameters as float32 arrays (bf16-representable for bf16 configs).

    Layouts: node_w [2^d-1, D], node_b [2^d-1], w1 [2^d, l, D], b1 [2^d, l],
    w2 [2^d, O, l], b2 [2^d, O]; nodes in breadth-first order
    (N_{m,n} at row 2^m - 1 + n).
    """
    D, O, l, nn, nl = cfg.D, cfg.O, cfg.leaf_width, cfg.n_nodes, cfg.n_leaves
    w = {
        "node_w": _normal(seed, _S_NODE_W, (nn, D), D ** -0.5),
        "node_b": (_normal(seed, _S_NODE_B, (nn,), cfg.node_bias_std)
                   if cfg.node_bias_std > 0 else np.zeros((nn,), np.float32)),
        "w1": _normal(seed, _S_W1, (nl, l, D), D ** -0.5),
        "b1": _normal(seed, _S_B1, (nl, l), LEAF_BIAS_STD),
        "w2": _normal(seed, _S_W2, (nl, O, l), l ** -0.5),
        "b2": _normal(seed, _S_B2, (nl, O), LEAF_BIAS_STD),
    }
    return {k: _store(cfg, v) for k, v in w.items()}


E4M3_MAX = 448.0


def e4m3_decode_table() -> np.ndarray:
    """float32 value of each of the 256 e4m3 codes (the library's conversion; the two NaN codes read as NaN)."""
    import torch
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    return codes.view(torch.float8_e4m3fn).to(torch.float32).numpy()


def quantize_e4m3(w: np.ndarray):
    """Storage encoding of leaf weights as 8-bit floats with one scale per leaf.

    w: float32 [n_leaves, ...].  Returns (codes uint8 like w, scales float32 [n_leaves], values float64 like w):
    scale_j = max|w_j| / 448 (1 for an all-zero leaf), code = the library's round-to-nearest-even e4m3 conversion of
    w / scale, values = decode(code) * scale in float64, i.e. exactly what the stored bytes and scales stand for.
    Both the oracle and the CUDA library are given these values (as float64 numbers, as codes and scales)."""
    import torch
    w = np.ascontiguousarray(w, dtype=np.float32)
    nl = w.shape[0]
    amax = np.abs(w.reshape(nl, -1)).max(axis=1)
    scales = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    scaled = w / scales.reshape((nl,) + (1,) * (w.ndim - 1))
    codes = torch.from_numpy(scaled).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    values = e4m3_decode_table().astype(np.float64)[codes] * scales.astype(np.float64).reshape((nl,) + (1,) * (w.ndim - 1))
    return codes, scales, values


def zipf_weights(n: int = N_CLUSTERS, s: float = ZIPF_S) -> np.ndarray:
    w = np.arange(1, n + 1, dtype=np.float64) ** (-s)
    return w / w.sum()


class TokenSource:
    """Batch of token rows plus the means to redraw individual rows."""

    def __init__(self, cfg: FFFConfig, seed: int = 0, B: Optional[int] = None):
        self.cfg, self.seed = cfg, seed
        self.B = cfg.B if B is None else int(B)
        D = cfg.D
        if cfg.x_kind == "clusters":
            self.centres = _rng(seed, _S_CENTRES).standard_normal(size=(N_CLUSTERS, D), dtype=np.float32)
            u = _rng(seed, _S_PICKS).random(size=self.B)
            self.cluster = np.minimum(np.searchsorted(np.cumsum(zipf_weights()), u), N_CLUSTERS - 1)
        else:
            self.centres = None
            self.cluster = None
        g = _rng(seed, _S_X).standard_normal(size=(self.B, D), dtype=np.float32)
        self.x = self._shape_rows(g, np.arange(self.B))

    def _shape_rows(self, g: np.ndarray, idx: np.ndarray) -> np.ndarray:
        kind = self.cfg.x_kind
        if kind == "normal":
            x = g
        elif kind == "layernorm":
            g64 = g.astype(np.float64)
            g64 -= g64.mean(axis=1, keepdims=True)
            g64 /= g64.std(axis=1, keepdims=True)
            x = g64.astype(np.float32)
        elif kind == "clusters":
            x = self.centres[self.cluster[idx]] + np.float32(CLUSTER_SIGMA) * g
        else:
            raise ValueError(f"unknown x_kind {kind!r}")
        return _store(self.cfg, x)

    def redraw(self, idx: np.ndarray, attempt: int) -> None:
        """Replace rows `idx` by fresh draws of the same kind (same cluster for mixtures)."""
        idx = np.asarray(idx, dtype=np.int64)
        if idx.size == 0:
            return
        g = _rng(self.seed, _S_REDRAW, attempt).standard_normal(size=(idx.size, self.cfg.D), dtype=np.float32)
        self.x[idx] = self._shape_rows(g, idx)


def enforce_margin(src: TokenSource,
                   margin_fn: Callable[[np.ndarray], np.ndarray],
                   margin: float = DEFAULT_MARGIN,
                   max_rounds: int = 64) -> int:
    """Redraw rows until `margin_fn(rows)` >= margin for every row.

    `margin_fn` maps a [n, D] float32 array to n non-negative floats (the
    smallest routing-logit magnitude met by each row); it is supplied by the
    caller.  Returns the number of rows that were redrawn at least once.
    """
    if src.cfg.depth == 0 or src.B == 0:
        return 0
    todo = np.arange(src.B)
    touched = 0
    for attempt in range(1, max_rounds + 1):
        m = np.asarray(margin_fn(src.x[todo]))
        bad = todo[m < margin]
        if bad.size == 0:
            return touched
        if attempt == 1:
            touched = int(bad.size)
        src.redraw(bad, attempt)
        todo = bad
    raise RuntimeError("margin resampling did not converge")
