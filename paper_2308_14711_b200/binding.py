"""ctypes binding of libfff.so: the same calls as include/fff.h, arguments marshalled only.

Every computation happens in the CUDA library.  If the library has not been
built (python -m paper_2308_14711_b200.build) loading fails with an error;
there is no fallback of any kind.

The module-level fff_* functions take raw device addresses (ints); `FFFLayer`
is a convenience wrapper that takes torch CUDA tensors, checks their dtype,
shape and contiguity, and passes their data_ptr().
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libfff.so")

FFF_OK = 0
STATUS_NAMES = {0: "FFF_OK", 1: "FFF_ERR_INVALID_ARG", 2: "FFF_ERR_UNSUPPORTED", 3: "FFF_ERR_ALLOC",
                4: "FFF_ERR_CUDA", 5: "FFF_ERR_DEVICE_TIMEOUT", 6: "FFF_ERR_BAD_HANDLE", 7: "FFF_ERR_TOO_LARGE"}
ACTIVATIONS = {"relu": 0, "gelu": 1, "gelu_tanh": 2, "silu": 3}
DTYPES = {"f32": 0, "bf16": 1}
PATHS = {"auto": 0, "warp": 1, "tensor": 2, "fused": 3}
TUNING = {"tcgen05_descent": 0, "tcgen05_grouped": 1, "tcgen05_leaf": 2, "cta_pairs": 3, "direct_lists": 4, "fused_small": 5, "group_tiles": 6}

# every symbol include/fff.h declares
EXPORTS = ["fff_create", "fff_create_w8", "fff_forward_infer", "fff_forward_train", "fff_forward_infer_host", "fff_destroy", "fff_reserve",
           "fff_set_path", "fff_set_tuning", "fff_tree_descent", "fff_leaf_bucketing", "fff_grouped_leaf_ff",
           "fff_debug_get_bucketing", "fff_get_last_status", "fff_capabilities", "fff_selftest_bounded_wait", "fff_last_launch_count", "fff_status_string",
           "fff_profile_begin", "fff_profile_end", "fff_profile_launches", "fff_profile_launch_name",
           "fff_leaf_bucketing_static", "fff_stack_create", "fff_stack_forward", "fff_stack_set_graph",
           "fff_stack_last_launch_count", "fff_stack_last_was_replay", "fff_stack_destroy"]


class FFFError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({status_string(status)})")


_lib = None


def lib():
    """Load libfff.so (once). Raises if it is missing: the CUDA library is the only implementation."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2308_14711_b200.build` "
                          "(needs nvcc); there is no CPU fallback")
    L = C.CDLL(LIB_PATH)
    vp, i64, ci = C.c_void_p, C.c_int64, C.c_int
    L.fff_create.argtypes = [C.POINTER(vp), ci, ci, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp]
    L.fff_forward_infer.argtypes = [vp, vp, vp, vp, i64, vp]
    L.fff_forward_infer_host.argtypes = [vp, vp, vp, vp, i64, vp]
    L.fff_destroy.argtypes = [vp]
    L.fff_reserve.argtypes = [vp, i64]
    L.fff_set_path.argtypes = [vp, ci]
    L.fff_set_tuning.argtypes = [vp, ci, ci]
    L.fff_create_w8.argtypes = [C.POINTER(vp), ci, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp]
    L.fff_capabilities.argtypes = [vp]
    L.fff_forward_train.argtypes = [vp, vp, vp, vp, vp, i64, vp]
    L.fff_stack_create.argtypes = [C.POINTER(vp), ci, C.POINTER(vp), ci, C.POINTER(vp), C.POINTER(vp), C.c_float, ci]
    L.fff_stack_forward.argtypes = [vp, vp, vp, vp, i64, vp]
    L.fff_stack_set_graph.argtypes = [vp, ci]
    L.fff_stack_last_launch_count.argtypes = [vp]
    L.fff_stack_last_was_replay.argtypes = [vp]
    L.fff_stack_destroy.argtypes = [vp]
    L.fff_selftest_bounded_wait.argtypes = [vp, i64, vp]
    L.fff_tree_descent.argtypes = [vp, vp, vp, i64, vp]
    L.fff_leaf_bucketing.argtypes = [vp, vp, vp, vp, i64, vp]
    L.fff_grouped_leaf_ff.argtypes = [vp, vp, vp, vp, vp, vp, i64, vp]
    L.fff_debug_get_bucketing.argtypes = [vp, vp, vp, vp]
    L.fff_get_last_status.argtypes = [vp]
    L.fff_last_launch_count.argtypes = [vp]
    L.fff_leaf_bucketing_static.argtypes = [vp, vp, vp, i64, ci, vp]
    L.fff_profile_begin.argtypes = [vp, ci]
    L.fff_profile_end.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(ci)]
    L.fff_profile_launches.argtypes = [vp]
    L.fff_profile_launch_name.argtypes = [vp, ci]
    for name in EXPORTS:
        getattr(L, name).restype = ci
    L.fff_profile_launch_name.restype = C.c_char_p
    L.fff_status_string.argtypes = [ci]
    L.fff_status_string.restype = C.c_char_p
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().fff_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != FFF_OK:
        raise FFFError(status, where)


# ---- raw calls: device addresses as ints, 0 / None for NULL ------------------------------------

def fff_create(D, O, depth, leaf_width, act, dtype, node_w, node_b, leaf_w1, leaf_b1, leaf_w2, leaf_b2) -> int:
    h = C.c_void_p()
    _check(lib().fff_create(C.byref(h), D, O, depth, leaf_width, act, dtype,
                            node_w, node_b, leaf_w1, leaf_b1, leaf_w2, leaf_b2), "fff_create")
    return h.value


def fff_forward_infer(h, x, y, leaf_idx, B, stream=None) -> None:
    _check(lib().fff_forward_infer(h, x, y, leaf_idx, B, stream), "fff_forward_infer")


def fff_forward_infer_host(h, x_host, y_host, leaf_idx_host, B, stream=None) -> None:
    _check(lib().fff_forward_infer_host(h, x_host, y_host, leaf_idx_host, B, stream), "fff_forward_infer_host")


def fff_destroy(h) -> None:
    _check(lib().fff_destroy(h), "fff_destroy")


def fff_reserve(h, max_B) -> None:
    _check(lib().fff_reserve(h, max_B), "fff_reserve")


def fff_set_path(h, path) -> None:
    _check(lib().fff_set_path(h, path), "fff_set_path")


def fff_set_tuning(h, key, value) -> None:
    _check(lib().fff_set_tuning(h, key, value), "fff_set_tuning")


def fff_tree_descent(h, x, leaf_idx, B, stream=None) -> None:
    _check(lib().fff_tree_descent(h, x, leaf_idx, B, stream), "fff_tree_descent")


def fff_leaf_bucketing(h, leaf_idx, offsets, perm, B, stream=None) -> None:
    _check(lib().fff_leaf_bucketing(h, leaf_idx, offsets, perm, B, stream), "fff_leaf_bucketing")


def fff_grouped_leaf_ff(h, x, leaf_idx, offsets, perm, y, B, stream=None) -> None:
    _check(lib().fff_grouped_leaf_ff(h, x, leaf_idx, offsets, perm, y, B, stream), "fff_grouped_leaf_ff")


def fff_debug_get_bucketing(h, perm, offsets, stream=None) -> None:
    _check(lib().fff_debug_get_bucketing(h, perm, offsets, stream), "fff_debug_get_bucketing")


def fff_get_last_status(h) -> int:
    return lib().fff_get_last_status(h)


def fff_selftest_bounded_wait(h, limit_cycles, stream=None) -> None:
    _check(lib().fff_selftest_bounded_wait(h, limit_cycles, stream), "fff_selftest_bounded_wait")


def fff_last_launch_count(h) -> int:
    return lib().fff_last_launch_count(h)


def fff_leaf_bucketing_static(leaf_idx, offsets, perm, B, depth, stream=None) -> None:
    """Handle-free, allocation-free bucketing (scratch compiled into the library; depth <= 16)."""
    _check(lib().fff_leaf_bucketing_static(leaf_idx, offsets, perm, B, depth, stream), "fff_leaf_bucketing_static")


def fff_profile_begin(h, max_steps) -> None:
    _check(lib().fff_profile_begin(h, max_steps), "fff_profile_begin")


def fff_profile_end(h):
    """Returns (list of (kernel name, mean ms) per launch position, number of recorded forwards)."""
    ms = (C.c_double * 16)()
    steps = C.c_int(0)
    _check(lib().fff_profile_end(h, ms, C.byref(steps)), "fff_profile_end")
    n = lib().fff_profile_launches(h)
    return [(lib().fff_profile_launch_name(h, i).decode(), ms[i]) for i in range(n)], steps.value


# ---- tensor-level convenience ------------------------------------------------------------------

def _torch():
    import torch
    return torch


def _ptr(t, dtype, shape, name):
    if t is None:
        return None
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: expected contiguous CUDA {dtype} tensor of shape {tuple(shape)}, "
                         f"got {t.dtype} {tuple(t.shape)} on {t.device}")
    return t.data_ptr()


class FFFLayer:
    """One FFF layer on the current CUDA device; tensors in, tensors out, all work in libfff.so."""

    def __init__(self, D: int, O: int, depth: int, leaf_width: int, activation: str, dtype: str,
                 node_w, node_b, w1, b1, w2, b2, path: str = "auto", w1_scale=None, w2_scale=None):
        """With w1_scale / w2_scale (float32 [2^d]) w1 and w2 are uint8 tensors of e4m3 codes (fff_create_w8)."""
        torch = _torch()
        self._h = None
        self.D, self.O, self.depth, self.l = D, O, depth, leaf_width
        self.n_leaves = 1 << depth
        self.tdtype = torch.float32 if dtype == "f32" else torch.bfloat16
        nn, nl = self.n_leaves - 1, self.n_leaves
        td = self.tdtype
        if w1_scale is not None:
            out = C.c_void_p()
            _check(lib().fff_create_w8(C.byref(out), D, O, depth, leaf_width, ACTIVATIONS[activation],
                                       _ptr(node_w, td, (nn, D), "node_w"), _ptr(node_b, td, (nn,), "node_b"),
                                       _ptr(w1, torch.uint8, (nl, leaf_width, D), "w1 codes"),
                                       _ptr(w1_scale, torch.float32, (nl,), "w1_scale"), _ptr(b1, td, (nl, leaf_width), "b1"),
                                       _ptr(w2, torch.uint8, (nl, O, leaf_width), "w2 codes"),
                                       _ptr(w2_scale, torch.float32, (nl,), "w2_scale"), _ptr(b2, td, (nl, O), "b2")),
                   "fff_create_w8")
            self._h = out.value
        else:
            self._h = fff_create(D, O, depth, leaf_width, ACTIVATIONS[activation], DTYPES[dtype],
                                 _ptr(node_w, td, (nn, D), "node_w"), _ptr(node_b, td, (nn,), "node_b"),
                                 _ptr(w1, td, (nl, leaf_width, D), "w1"), _ptr(b1, td, (nl, leaf_width), "b1"),
                                 _ptr(w2, td, (nl, O, leaf_width), "w2"), _ptr(b2, td, (nl, O), "b2"))
        if path != "auto":
            self.set_path(path)

    @property
    def handle(self) -> int:
        return self._h

    def close(self) -> None:
        if getattr(self, "_h", None):
            h, self._h = self._h, None
            fff_destroy(h)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _stream(self, stream):
        s = stream if stream is not None else _torch().cuda.current_stream()
        return s.cuda_stream

    def reserve(self, max_B: int) -> None:
        fff_reserve(self._h, max_B)

    def set_path(self, path: str) -> None:
        fff_set_path(self._h, PATHS[path])

    def capabilities(self) -> int:
        """Bit set of FFF_CAP_*: the kernel families this layer's shapes admit."""
        return lib().fff_capabilities(self._h)

    def set_tuning(self, key: str, on: bool) -> None:
        """Switch between kernels that compute the same thing (keys of TUNING; all on by default)."""
        fff_set_tuning(self._h, TUNING[key], 1 if on else 0)

    def forward_infer(self, x, y=None, leaf_idx=None, want_leaf_idx: bool = True, stream=None):
        torch = _torch()
        B = x.shape[0]
        if y is None:
            y = torch.empty((B, self.O), dtype=self.tdtype, device=x.device)
        if leaf_idx is None and want_leaf_idx:
            leaf_idx = torch.empty((B,), dtype=torch.int32, device=x.device)
        fff_forward_infer(self._h, _ptr(x, self.tdtype, (B, self.D), "x"), _ptr(y, self.tdtype, (B, self.O), "y"),
                          _ptr(leaf_idx, torch.int32, (B,), "leaf_idx"), B, self._stream(stream))
        return y, leaf_idx

    def forward_train(self, x, want_mixture: bool = True, want_entropy: bool = True, stream=None):
        """FORWARD_T: returns (y, mixture weights float32 [B, 2^d] or None, node entropies float32 [2^d - 1] or None)."""
        torch = _torch()
        B = x.shape[0]
        y = torch.empty((B, self.O), dtype=self.tdtype, device=x.device)
        mix = torch.empty((B, self.n_leaves), dtype=torch.float32, device=x.device) if want_mixture else None
        ent = torch.empty((max(self.n_leaves - 1, 1),), dtype=torch.float32, device=x.device) if want_entropy else None
        _check(lib().fff_forward_train(self._h, _ptr(x, self.tdtype, (B, self.D), "x"), y.data_ptr(),
                                       None if mix is None else mix.data_ptr(), None if ent is None else ent.data_ptr(), B,
                                       self._stream(stream)), "fff_forward_train")
        return y, mix, (None if ent is None else ent[:self.n_leaves - 1])

    def forward_infer_host(self, x_host, y_host, leaf_idx_host=None, stream=None) -> None:
        """x_host / y_host / leaf_idx_host: contiguous CPU tensors (pinned for full copy speed)."""
        B = x_host.shape[0]
        assert not x_host.is_cuda and not y_host.is_cuda and x_host.is_contiguous() and y_host.is_contiguous()
        assert x_host.dtype == self.tdtype and y_host.dtype == self.tdtype
        assert tuple(x_host.shape) == (B, self.D) and tuple(y_host.shape) == (B, self.O)
        fff_forward_infer_host(self._h, x_host.data_ptr(), y_host.data_ptr(),
                               None if leaf_idx_host is None else leaf_idx_host.data_ptr(), B, self._stream(stream))

    def tree_descent(self, x, leaf_idx=None, stream=None):
        torch = _torch()
        B = x.shape[0]
        if leaf_idx is None:
            leaf_idx = torch.empty((B,), dtype=torch.int32, device=x.device)
        fff_tree_descent(self._h, _ptr(x, self.tdtype, (B, self.D), "x"), _ptr(leaf_idx, torch.int32, (B,), "leaf_idx"),
                         B, self._stream(stream))
        return leaf_idx

    def leaf_bucketing(self, leaf_idx, stream=None):
        torch = _torch()
        B = leaf_idx.shape[0]
        offsets = torch.empty((self.n_leaves + 1,), dtype=torch.int32, device=leaf_idx.device)
        perm = torch.empty((B,), dtype=torch.int32, device=leaf_idx.device)
        fff_leaf_bucketing(self._h, _ptr(leaf_idx, torch.int32, (B,), "leaf_idx"), offsets.data_ptr(), perm.data_ptr(),
                           B, self._stream(stream))
        return offsets, perm

    def grouped_leaf_ff(self, x, leaf_idx, offsets, perm, y=None, stream=None):
        torch = _torch()
        B = x.shape[0]
        if y is None:
            y = torch.empty((B, self.O), dtype=self.tdtype, device=x.device)
        fff_grouped_leaf_ff(self._h, _ptr(x, self.tdtype, (B, self.D), "x"),
                            _ptr(leaf_idx, torch.int32, (B,), "leaf_idx"),
                            _ptr(offsets, torch.int32, (self.n_leaves + 1,), "offsets"),
                            _ptr(perm, torch.int32, (B,), "perm"), _ptr(y, self.tdtype, (B, self.O), "y"),
                            B, self._stream(stream))
        return y

    def last_bucketing(self, B: int, stream=None):
        torch = _torch()
        perm = torch.empty((B,), dtype=torch.int32, device="cuda")
        offsets = torch.empty((self.n_leaves + 1,), dtype=torch.int32, device="cuda")
        fff_debug_get_bucketing(self._h, perm.data_ptr(), offsets.data_ptr(), self._stream(stream))
        return offsets, perm

    def profile_begin(self, max_steps: int) -> None:
        fff_profile_begin(self._h, max_steps)

    def profile_end(self):
        return fff_profile_end(self._h)

    def last_status(self) -> int:
        return fff_get_last_status(self._h)

    def last_launch_count(self) -> int:
        return fff_last_launch_count(self._h)


class FFFStack:
    """Several FFFLayer objects of one width behind one handle: optional layer normalisation in front of every
    layer, optional residual connections, optional CUDA-graph replay.  The layers stay alive with the stack."""

    def __init__(self, layers, layer_norm: bool = True, gammas=None, betas=None, eps: float = 1e-5, residual: bool = True):
        torch = _torch()
        self._s = None
        self.layers = list(layers)
        n = len(self.layers)
        self.D = self.layers[0].D
        self.tdtype = self.layers[0].tdtype
        hs = (C.c_void_p * n)(*[l.handle for l in self.layers])

        def ptrs(vs):
            if vs is None:
                return None
            assert len(vs) == n
            return (C.c_void_p * n)(*[None if v is None else _ptr(v, self.tdtype, (self.D,), "layer-norm vector") for v in vs])
        out = C.c_void_p()
        _check(lib().fff_stack_create(C.byref(out), n, hs, 1 if layer_norm else 0, ptrs(gammas), ptrs(betas), eps,
                                      1 if residual else 0), "fff_stack_create")
        self._s = out.value

    def close(self) -> None:
        if getattr(self, "_s", None):
            s, self._s = self._s, None
            _check(lib().fff_stack_destroy(s), "fff_stack_destroy")

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_graph(self, on: bool) -> None:
        _check(lib().fff_stack_set_graph(self._s, 1 if on else 0), "fff_stack_set_graph")

    def forward(self, x, y=None, leaf_idx=None, want_leaf_idx: bool = True, stream=None):
        torch = _torch()
        B = x.shape[0]
        if y is None:
            y = torch.empty((B, self.D), dtype=self.tdtype, device=x.device)
        if leaf_idx is None and want_leaf_idx:
            leaf_idx = torch.empty((len(self.layers), B), dtype=torch.int32, device=x.device)
        st = (stream if stream is not None else torch.cuda.current_stream()).cuda_stream
        _check(lib().fff_stack_forward(self._s, _ptr(x, self.tdtype, (B, self.D), "x"), _ptr(y, self.tdtype, (B, self.D), "y"),
                                       _ptr(leaf_idx, torch.int32, (len(self.layers), B), "leaf_idx"), B, st), "fff_stack_forward")
        return y, leaf_idx

    def last_launch_count(self) -> int:
        return lib().fff_stack_last_launch_count(self._s)

    def last_was_replay(self) -> bool:
        return lib().fff_stack_last_was_replay(self._s) == 1
