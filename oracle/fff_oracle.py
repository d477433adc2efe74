"""ctypes front end of the float64 C oracle (test infrastructure only).

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import
this module.  Every function widens its inputs to float64 and calls the plain C
loops in fff_oracle.c; nothing here is shared with the CUDA path.
"""
from __future__ import annotations

import ctypes as C
import threading
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Optional, Tuple

import numpy as np

from . import build as _build

ACT = {"relu": 0, "gelu": 1, "gelu_tanh": 2, "silu": 3}

_lib = None
_dp = C.POINTER(C.c_double)
_ip = C.POINTER(C.c_int32)
_lp = C.POINTER(C.c_long)


_lib_lock = threading.Lock()


def lib():
    global _lib
    if _lib is None:
        with _lib_lock:
            if _lib is None:
                _lib = _load()
    return _lib


def _load():
    L = C.CDLL(_build.build())
    L.fff_oracle_descend.argtypes = [C.c_int, C.c_int, _dp, _dp, _dp, C.c_long, C.c_long, _ip, _dp, _lp]
    L.fff_oracle_descend.restype = None
    L.fff_oracle_forward_i.argtypes = [C.c_int] * 5 + [_dp] * 7 + [C.c_long, C.c_long, _dp, _ip, _lp, _lp]
    L.fff_oracle_forward_i.restype = None
    L.fff_oracle_forward_t.argtypes = [C.c_int] * 5 + [_dp] * 7 + [C.c_long, _dp]
    L.fff_oracle_mixture_weights.restype = None
    L.fff_oracle_mixture_weights.argtypes = [C.c_int, C.c_int, _dp, _dp, _dp, C.c_long, C.c_long, _dp]
    L.fff_oracle_node_entropy.restype = None
    L.fff_oracle_node_entropy.argtypes = [C.c_int, C.c_int, _dp, _dp, _dp, C.c_long, _dp]
    L.fff_oracle_forward_t.restype = None
    L.fff_oracle_forward_all_leaves_masked.argtypes = [C.c_int] * 5 + [_dp] * 5 + [C.c_long, _ip, _dp]
    L.fff_oracle_forward_all_leaves_masked.restype = None
    L.fff_oracle_brute_force_leaf.argtypes = [C.c_int, C.c_int, _dp, _dp, _dp, _ip]
    L.fff_oracle_brute_force_leaf.restype = C.c_int
    L.fff_oracle_bucket.argtypes = [_ip, C.c_long, C.c_long, _ip, _ip]
    L.fff_oracle_bucket.restype = None
    for name in ("training_size", "inference_size"):
        f = getattr(L, "fff_oracle_" + name)
        f.argtypes = [C.c_int] * 3
        f.restype = C.c_long
    L.fff_oracle_training_width.argtypes = [C.c_int, C.c_int]
    L.fff_oracle_training_width.restype = C.c_long
    L.fff_oracle_inference_width.argtypes = [C.c_int]
    L.fff_oracle_inference_width.restype = C.c_long
    return L


def _d(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a: np.ndarray):
    return a.ctypes.data_as(_dp)


class Net:
    """FFF parameters widened to float64 once, so repeated calls do not re-convert."""

    def __init__(self, D: int, O: int, depth: int, leaf_width: int, activation: str,
                 node_w, node_b, w1, b1, w2, b2):
        self.D, self.O, self.depth, self.l = int(D), int(O), int(depth), int(leaf_width)
        self.act = ACT[activation]
        nn, nl = (1 << depth) - 1, 1 << depth
        self.node_w = _d(node_w if node_w is not None else np.zeros((nn, D))).reshape(nn, D)
        self.node_b = _d(node_b if node_b is not None else np.zeros((nn,))).reshape(nn)
        self.w1 = _d(w1).reshape(nl, self.l, D)
        self.b1 = _d(b1 if b1 is not None else np.zeros((nl, self.l))).reshape(nl, self.l)
        self.w2 = _d(w2).reshape(nl, O, self.l)
        self.b2 = _d(b2 if b2 is not None else np.zeros((nl, O))).reshape(nl, O)

    @classmethod
    def from_config(cls, cfg, weights: Dict[str, np.ndarray]) -> "Net":
        return cls(cfg.D, cfg.O, cfg.depth, cfg.leaf_width, cfg.activation, **weights)

    def _head(self):
        return (self.D, self.O, self.depth, self.l, self.act)

    def _params(self):
        return tuple(_p(a) for a in (self.node_w, self.node_b, self.w1, self.b1, self.w2, self.b2))


def _split(B: int, threads: int):
    threads = max(1, min(int(threads), B if B > 0 else 1))
    edges = np.linspace(0, B, threads + 1).astype(np.int64)
    return [(int(a), int(b)) for a, b in zip(edges[:-1], edges[1:]) if b > a]


def descend(net: Net, x, threads: int = 1) -> Tuple[np.ndarray, np.ndarray, int]:
    """Hard descent. Returns (leaf_idx int32[B], min |logit| on the path float64[B], node evaluations)."""
    x = _d(x).reshape(-1, net.D)
    B = x.shape[0]
    leaf = np.zeros(B, np.int32)
    mn = np.full(B, np.inf)
    parts = _split(B, threads)
    counts = [C.c_long(0) for _ in parts]

    def run(i):
        a, b = parts[i]
        lib().fff_oracle_descend(net.D, net.depth, _p(net.node_w), _p(net.node_b), _p(x), a, b,
                                 leaf.ctypes.data_as(_ip), _p(mn), C.byref(counts[i]))
    _run(run, len(parts))
    return leaf, mn, sum(c.value for c in counts)


def path_margin(net: Net, x, threads: int = 1) -> np.ndarray:
    """Smallest |node logit| along each token's path (float64)."""
    return descend(net, x, threads)[1]


def forward_i(net: Net, x, threads: int = 1, counters: Optional[dict] = None) -> Tuple[np.ndarray, np.ndarray]:
    """FORWARD_I. Returns (y float64[B,O], leaf_idx int32[B])."""
    x = _d(x).reshape(-1, net.D)
    B = x.shape[0]
    y = np.zeros((B, net.O))
    leaf = np.zeros(B, np.int32)
    parts = _split(B, threads)
    ne = [C.c_long(0) for _ in parts]
    le = [C.c_long(0) for _ in parts]

    def run(i):
        a, b = parts[i]
        lib().fff_oracle_forward_i(*net._head(), *net._params(), _p(x), a, b, _p(y),
                                   leaf.ctypes.data_as(_ip), C.byref(ne[i]), C.byref(le[i]))
    _run(run, len(parts))
    if counters is not None:
        counters["node_evals"] = sum(c.value for c in ne)
        counters["leaf_evals"] = sum(c.value for c in le)
    return y, leaf


def _run(fn, n: int) -> None:
    if n <= 1:
        for i in range(n):
            fn(i)
        return
    with ThreadPoolExecutor(max_workers=n) as ex:   # ctypes releases the GIL during the C call
        list(ex.map(fn, range(n)))


def forward_t(net: Net, x) -> np.ndarray:
    """FORWARD_T (soft mixture over all leaves); small trees only."""
    x = _d(x).reshape(-1, net.D)
    y = np.zeros((x.shape[0], net.O))
    lib().fff_oracle_forward_t(*net._head(), *net._params(), _p(x), x.shape[0], _p(y))
    return y


def forward_t_rows(net: Net, x, threads: int = 1) -> np.ndarray:
    """FORWARD_T with the token loop split over threads (tokens are independent)."""
    x = _d(x).reshape(-1, net.D)
    B = x.shape[0]
    y = np.zeros((B, net.O))
    parts = _split(B, threads)

    def run(i):
        a, b = parts[i]
        lib().fff_oracle_forward_t(*net._head(), *net._params(), _p(x[a:b]), b - a, _p(y[a:b]))
    _run(run, len(parts))
    return y


def mixture_weights(net: Net, x, threads: int = 1) -> np.ndarray:
    """Weight of every leaf in FORWARD_T's mixture, float64 [B, 2^d]."""
    x = _d(x).reshape(-1, net.D)
    B = x.shape[0]
    mix = np.zeros((B, 1 << net.depth))
    parts = _split(B, threads)

    def run(i):
        a, b = parts[i]
        lib().fff_oracle_mixture_weights(net.D, net.depth, _p(net.node_w), _p(net.node_b), _p(x), a, b, _p(mix))
    _run(run, len(parts))
    return mix


def node_entropy(net: Net, x) -> np.ndarray:
    """Batch mean of the entropy (nats) of every node's choice, float64 [2^d - 1]."""
    x = _d(x).reshape(-1, net.D)
    ent = np.zeros(max((1 << net.depth) - 1, 1))
    lib().fff_oracle_node_entropy(net.D, net.depth, _p(net.node_w), _p(net.node_b), _p(x), x.shape[0], _p(ent))
    return ent[:(1 << net.depth) - 1]


def forward_all_leaves_masked(net: Net, x, leaf_idx) -> np.ndarray:
    x = _d(x).reshape(-1, net.D)
    leaf_idx = np.ascontiguousarray(leaf_idx, dtype=np.int32)
    y = np.zeros((x.shape[0], net.O))
    lib().fff_oracle_forward_all_leaves_masked(*net._head(), *net._params()[2:], _p(x), x.shape[0],
                                               leaf_idx.ctypes.data_as(_ip), _p(y))
    return y


def brute_force_leaf(net: Net, x_row) -> Tuple[int, int]:
    """(number of leaves whose region contains x_row, the last such leaf)."""
    x_row = _d(x_row).reshape(net.D)
    leaf = C.c_int32(-1)
    hits = lib().fff_oracle_brute_force_leaf(net.D, net.depth, _p(net.node_w), _p(net.node_b), _p(x_row),
                                             C.byref(leaf))
    return hits, leaf.value


def bucket(leaf_idx, n_leaves: int) -> Tuple[np.ndarray, np.ndarray]:
    """Stable counting sort of token ids by leaf. Returns (offsets int32[n_leaves+1], perm int32[B])."""
    leaf_idx = np.ascontiguousarray(leaf_idx, dtype=np.int32)
    B = leaf_idx.shape[0]
    offsets = np.zeros(n_leaves + 1, np.int32)
    perm = np.zeros(B, np.int32)
    lib().fff_oracle_bucket(leaf_idx.ctypes.data_as(_ip), B, n_leaves,
                            offsets.ctypes.data_as(_ip), perm.ctypes.data_as(_ip))
    return offsets, perm


def training_size(d: int, n: int, l: int) -> int:
    return lib().fff_oracle_training_size(d, n, l)


def inference_size(d: int, n: int, l: int) -> int:
    return lib().fff_oracle_inference_size(d, n, l)


def training_width(d: int, l: int) -> int:
    return lib().fff_oracle_training_width(d, l)


def inference_width(l: int) -> int:
    return lib().fff_oracle_inference_width(l)
