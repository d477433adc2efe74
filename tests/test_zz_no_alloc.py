"""The allocation-free bucketing entry point against the handle-based one.

fff_leaf_bucketing_static is for callers that may not allocate device memory (hosts that own all device
memory, allocation-accounting windows, latency-critical loops); its counters live in an array compiled into
the library instead of a handle's workspace.  It must return exactly what fff_leaf_bucketing returns
(integer results: bit-exact), also when the shared array still holds the counts of an earlier, different
call.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2308_14711_b200 import binding, workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def _keys(B, depth, seed, skew):
    rng = np.random.default_rng(seed)
    nl = 1 << depth
    k = np.minimum(rng.zipf(1.3, size=B) - 1, nl - 1) if skew else rng.integers(0, nl, size=B)
    return torch.from_numpy(k.astype(np.int32)).cuda()


def _handle_based(depth, keys):
    cfg = wl.FFFConfig("z", 8, 8, depth, 1, "relu", "f32", 1)
    layer = util.make_layer(util.Case(cfg, wl.make_weights(cfg, 0), None, None, 0))
    off, perm = layer.leaf_bucketing(keys)
    torch.cuda.synchronize()
    layer.close()
    return off, perm


def _static(depth, keys):
    B = keys.shape[0]
    off = torch.full(((1 << depth) + 1,), -7, dtype=torch.int32, device="cuda")
    perm = torch.full((max(B, 1),), -7, dtype=torch.int32, device="cuda")[:B]
    binding.fff_leaf_bucketing_static(keys.data_ptr(), off.data_ptr(), perm.data_ptr(), B, depth,
                                      torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return off, perm


def test_static_bucketing_equals_handle_bucketing_on_consecutive_calls():
    # two calls in a row on the shared array: a large skewed one, then a smaller one with fewer bins whose
    # counters overlap the first call's; then the first again
    calls = [(60000, 11, True), (5000, 6, False), (60000, 11, True), (0, 3, False), (777, 16, False)]
    for i, (B, depth, skew) in enumerate(calls):
        keys = _keys(B, depth, seed=i, skew=skew)
        off_ref, perm_ref = _handle_based(depth, keys)
        off, perm = _static(depth, keys)
        assert torch.equal(off, off_ref), f"offsets differ on call {i}"
        assert torch.equal(perm, perm_ref), f"perm differs on call {i}"
        assert int(off[-1]) == B


def test_static_bucketing_rejects_sizes_beyond_its_capacity():
    L = binding.lib()
    one = torch.zeros(4, dtype=torch.int32, device="cuda")
    assert L.fff_leaf_bucketing_static(one.data_ptr(), one.data_ptr(), one.data_ptr(), 1, 17, None) == 7
    assert L.fff_leaf_bucketing_static(one.data_ptr(), one.data_ptr(), one.data_ptr(), 2 ** 31, 3, None) == 7
    assert L.fff_leaf_bucketing_static(one.data_ptr(), one.data_ptr(), one.data_ptr(), -1, 3, None) == 1
    assert L.fff_leaf_bucketing_static(one.data_ptr(), None, one.data_ptr(), 1, 1, None) == 1
    assert "static scratch" in binding.status_string(7)
    torch.cuda.synchronize()
