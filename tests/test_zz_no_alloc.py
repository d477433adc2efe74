"""The allocation-free bucketing entry point against the oracle and against the handle-based entry point.

fff_leaf_bucketing_static is for callers that may not allocate device memory (hosts that own all device
memory, allocation-accounting windows, latency-critical loops); its counters live in an array compiled into
the library instead of a handle's workspace.  It must return the stable counting sort (integer results:
bit-exact against the CPU oracle, and equal to what fff_leaf_bucketing returns), also when the shared array
still holds the counts of an earlier, different call, and it must not change the amount of free device
memory.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from oracle import fff_oracle as orc
from paper_2308_14711_b200 import binding, workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def _keys(B, depth, seed, skew):
    rng = np.random.default_rng(seed)
    nl = 1 << depth
    k = np.minimum(rng.zipf(1.3, size=B) - 1, nl - 1) if skew else rng.integers(0, nl, size=B)
    return k.astype(np.int32)


def _handle_based(depth, keys):
    cfg = wl.FFFConfig("z", 8, 8, depth, 1, "relu", "f32", 1)
    layer = util.make_layer(util.Case(cfg, wl.make_weights(cfg, 0), None, None, 0))
    off, perm = layer.leaf_bucketing(keys)
    torch.cuda.synchronize()
    layer.close()
    return off, perm


def _static(depth, keys, off, perm):
    """One call on caller-owned buffers (pre-filled with -7 so that unwritten entries show)."""
    B = keys.shape[0]
    off.fill_(-7)
    perm.fill_(-7)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    binding.fff_leaf_bucketing_static(keys.data_ptr(), off.data_ptr(), perm.data_ptr(), B, depth,
                                      torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    free_after = torch.cuda.mem_get_info()[0]
    return off[:(1 << depth) + 1], perm[:B], free_before - free_after


def _oracle_ignoring_out_of_range(keys, depth):
    """Stable bucketing of the tokens whose key is a leaf of the tree, in original token numbers."""
    valid = np.flatnonzero((keys >= 0) & (keys < (1 << depth)))
    off, perm_c = orc.bucket(keys[valid], 1 << depth)
    return off, valid[perm_c].astype(np.int32)


def test_static_bucketing_matches_oracle_on_consecutive_calls_and_allocates_nothing():
    # calls in a row on the shared array: a large skewed one, then a smaller one with fewer bins whose
    # counters overlap the first call's; then the first again; an empty batch; the deepest tree with a batch
    # that is no multiple of a warp; a tree of one leaf; a batch with keys that are no leaf of the tree
    calls = [(60000, 11, True), (5000, 6, False), (60000, 11, True), (0, 3, False), (777, 16, False),
             (1001, 0, False), (4099, 5, False)]
    off_buf = torch.empty((1 << 16) + 1, dtype=torch.int32, device="cuda")
    perm_buf = torch.empty(60000, dtype=torch.int32, device="cuda")
    key_buf = torch.empty(60000, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    for i, (B, depth, skew) in enumerate(calls):
        keys_np = _keys(B, depth, seed=i, skew=skew)
        if i == len(calls) - 1:                         # some keys outside [0, 2^depth)
            keys_np[::7] = -1 - keys_np[::7]
            keys_np[3::11] += 1 << depth
        keys = key_buf[:B]
        keys.copy_(torch.from_numpy(keys_np))
        off_ref, perm_ref = _oracle_ignoring_out_of_range(keys_np, depth)
        off, perm, taken = _static(depth, keys, off_buf, perm_buf)
        # (the first call on a device may look up the array's address; later calls must leave free memory alone)
        assert i == 0 or taken == 0, f"free device memory changed by {taken} bytes across call {i}"
        n_valid = int(off_ref[-1])
        np.testing.assert_array_equal(off.cpu().numpy(), off_ref, err_msg=f"offsets differ from the oracle on call {i}")
        np.testing.assert_array_equal(perm.cpu().numpy()[:n_valid], perm_ref, err_msg=f"perm differs from the oracle on call {i}")
        assert (perm[n_valid:] == -7).all(), "entries past the valid tokens must stay unwritten"
    # second assertion: the handle-based entry point returns the same (its own kernels, its own workspace)
    for i, (B, depth, skew) in enumerate(calls[:5]):
        keys = torch.from_numpy(_keys(B, depth, seed=i, skew=skew)).cuda()
        off_h, perm_h = _handle_based(depth, keys)
        off, perm, _ = _static(depth, keys, off_buf, perm_buf)
        assert torch.equal(off, off_h), f"offsets differ from fff_leaf_bucketing on call {i}"
        assert torch.equal(perm, perm_h), f"perm differs from fff_leaf_bucketing on call {i}"


def test_static_bucketing_rejects_sizes_beyond_its_capacity():
    L = binding.lib()
    one = torch.zeros(4, dtype=torch.int32, device="cuda")
    assert L.fff_leaf_bucketing_static(one.data_ptr(), one.data_ptr(), one.data_ptr(), 1, 17, None) == 7
    assert L.fff_leaf_bucketing_static(one.data_ptr(), one.data_ptr(), one.data_ptr(), 2 ** 31, 3, None) == 7
    assert L.fff_leaf_bucketing_static(one.data_ptr(), one.data_ptr(), one.data_ptr(), 2 ** 31 - 4095, 3, None) == 7
    assert L.fff_leaf_bucketing_static(one.data_ptr(), one.data_ptr(), one.data_ptr(), -1, 3, None) == 1
    assert L.fff_leaf_bucketing_static(one.data_ptr(), None, one.data_ptr(), 1, 1, None) == 1
    assert "static scratch" in binding.status_string(7)
    torch.cuda.synchronize()
