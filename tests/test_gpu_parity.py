"""GPU parity: the CUDA library, called through its C ABI, against the float64 CPU oracle.

Integer results (leaf indices, bucket offsets, bucket permutation) must be bit-exact.
Outputs must satisfy  |err| <= 1e-5 (1 + |ref|)  for float32 layers and
|err| <= 2e-2 (1 + |ref|)  with relative L2 error <= 1e-2  for bf16 layers.
Inputs are margin-enforced (no routing logit within 1e-2 of zero), so the routing decision
cannot depend on summation order.
"""
import numpy as np
import pytest
import torch

from oracle import fff_oracle as orc
from paper_2308_14711_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu

PATHS = ["auto", "warp", "tensor", "fused"]


def layer_on_path(case, path):
    """Layer pinned to a kernel family; skips when the shapes cannot run on it."""
    from paper_2308_14711_b200.binding import FFFError
    try:
        return util.make_layer(case, path)
    except FFFError as e:
        if e.status == 2:
            pytest.skip(f"{case.cfg.name}: shapes not eligible for the {path} path")
        raise


def small_cfgs():
    C = wl.FFFConfig
    return [
        # ragged D (not a multiple of the vector width), tiny O, float32
        C("f32_ragged", 50, 3, 3, 5, "relu", "f32", 333, "normal", node_bias_std=0.3),
        C("f32_mnistlike", 784, 10, 3, 32, "relu", "f32", 517, "normal"),
        C("f32_gelu_d0", 64, 16, 0, 8, "gelu", "f32", 100, "normal"),
        C("f32_d1", 32, 32, 1, 4, "gelu", "f32", 65, "normal", node_bias_std=0.5),
        # bf16: several tiles and a ragged tail, l below / at / above the MMA granule
        C("bf16_l12", 768, 768, 4, 12, "gelu", "bf16", 1500, "layernorm"),
        C("bf16_l32", 256, 128, 6, 32, "gelu", "bf16", 3001, "normal"),
        C("bf16_l1_deep", 128, 64, 10, 1, "gelu", "bf16", 700, "normal"),
        C("bf16_skew", 128, 256, 7, 16, "relu", "bf16", 4099, "clusters"),
        C("bf16_ragged", 100, 36, 3, 7, "gelu", "bf16", 257, "normal", node_bias_std=0.2),
        C("bf16_d0", 128, 128, 0, 48, "gelu", "bf16", 300, "normal"),
        C("bf16_one_token", 64, 64, 5, 16, "gelu", "bf16", 1, "normal"),
        C("bf16_l40", 512, 520, 2, 40, "relu", "bf16", 999, "normal"),
        # O not a multiple of the 128-column output pieces; fewer tokens than one 128-row tile
        C("bf16_o208", 384, 208, 5, 20, "gelu", "bf16", 2000, "normal"),
        C("bf16_tiny_batch", 128, 144, 3, 16, "relu", "bf16", 37, "normal", node_bias_std=0.2),
        # the other two leaf activations: float32 (one-launch and warp kernels) and bf16 (tensor-core epilogues, l below
        # and at the padded width, thin buckets; warp kernels)
        C("f32_silu", 96, 12, 3, 16, "silu", "f32", 700, "normal", node_bias_std=0.2),
        C("f32_gelu_tanh", 200, 24, 2, 32, "gelu_tanh", "f32", 450, "normal"),
        C("bf16_silu_l12", 256, 128, 5, 12, "silu", "bf16", 2500, "normal"),
        C("bf16_gelu_tanh_l32", 128, 256, 6, 32, "gelu_tanh", "bf16", 3001, "clusters"),
        # eight levels in one dense stage (255 nodes), small batch
        C("bf16_d8_small", 256, 64, 8, 8, "gelu", "bf16", 5000, "layernorm"),
        # more 128-token tiles than SMs: the first stage runs on CTA pairs (127 nodes, odd number of tiles)
        C("bf16_d7_pairs", 128, 64, 7, 8, "relu", "bf16", 20001, "normal"),
    ]


@pytest.fixture(scope="module", params=small_cfgs(), ids=lambda c: c.name)
def small_case(request):
    case = util.make_case(request.param, seed=1)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    return case, y_ref, leaf_ref


@pytest.mark.parametrize("path", PATHS)
def test_forward_matches_oracle_elementwise(small_case, path):
    case, y_ref, leaf_ref = small_case
    cfg = case.cfg
    layer = layer_on_path(case, path)
    x = util.to_device(case.x, cfg.dtype)
    y, leaf = layer.forward_infer(x)
    torch.cuda.synchronize()
    assert layer.last_launch_count() > 0
    np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
    off_ref, perm_ref = orc.bucket(leaf_ref, cfg.n_leaves)
    off, perm = layer.last_bucketing(cfg.B)
    np.testing.assert_array_equal(off.cpu().numpy(), off_ref)
    np.testing.assert_array_equal(perm.cpu().numpy(), perm_ref)
    util.check_outputs(y, y_ref, cfg.dtype)
    assert layer.last_status() == 0
    # leaf_idx is optional
    y2, none = layer.forward_infer(x, want_leaf_idx=False)
    assert none is None
    assert torch.equal(y2, y)
    layer.close()


@pytest.mark.parametrize("path", PATHS)
def test_stage_entry_points_match_oracle(small_case, path):
    case, y_ref, leaf_ref = small_case
    cfg = case.cfg
    layer = layer_on_path(case, path)
    x = util.to_device(case.x, cfg.dtype)
    leaf = layer.tree_descent(x)
    np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
    off, perm = layer.leaf_bucketing(leaf)
    off_ref, perm_ref = orc.bucket(leaf_ref, cfg.n_leaves)
    np.testing.assert_array_equal(off.cpu().numpy(), off_ref)
    np.testing.assert_array_equal(perm.cpu().numpy(), perm_ref)
    y = layer.grouped_leaf_ff(x, leaf, off, perm)
    util.check_outputs(y, y_ref, cfg.dtype)
    layer.close()


def test_runs_are_bit_reproducible(small_case):
    case, _, _ = small_case
    layer = util.make_layer(case)
    x = util.to_device(case.x, case.cfg.dtype)
    y1, l1 = layer.forward_infer(x)
    y2, l2 = layer.forward_infer(x)
    assert torch.equal(y1, y2) and torch.equal(l1, l2)
    layer.close()


@pytest.mark.parametrize("B,depth,kind", [(0, 3, "uniform"), (1, 0, "uniform"), (31, 2, "uniform"), (4097, 5, "uniform"),
                                          (70001, 11, "uniform"), (50000, 11, "one_bin"), (50000, 11, "zipf"),
                                          (20000, 15, "uniform"), (3000, 15, "each_own"), (100000, 3, "uniform"),
                                          (9999, 16, "zipf")])
def test_bucketing_is_the_stable_counting_sort(B, depth, kind):
    nl = 1 << depth
    rng = np.random.default_rng(B + depth)
    if kind == "uniform":
        keys = rng.integers(0, nl, size=B)
    elif kind == "one_bin":
        keys = np.full(B, nl - 3)
    elif kind == "each_own":
        keys = rng.permutation(nl)[:B]
    else:
        keys = np.minimum(rng.zipf(1.3, size=B) - 1, nl - 1)
    keys = keys.astype(np.int32)
    cfg = wl.FFFConfig("b", 8, 8, depth, 1, "relu", "f32", max(B, 1))
    w = wl.make_weights(cfg, 0)
    case = util.Case(cfg, w, None, None, 0)
    layer = util.make_layer(case)
    dkeys = torch.from_numpy(keys).cuda()
    for _ in range(2):      # twice: the histogram buffers alternate between calls
        off, perm = layer.leaf_bucketing(dkeys)
        off_ref, perm_ref = orc.bucket(keys, nl)
        np.testing.assert_array_equal(off.cpu().numpy(), off_ref)
        np.testing.assert_array_equal(perm.cpu().numpy(), perm_ref)
    layer.close()


def test_host_buffer_entry_point(small_case):
    case, y_ref, leaf_ref = small_case
    cfg = case.cfg
    layer = util.make_layer(case)
    td = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    xh = torch.from_numpy(case.x).to(td).pin_memory()
    yh = torch.empty((cfg.B, cfg.O), dtype=td).pin_memory()
    lh = torch.empty((cfg.B,), dtype=torch.int32).pin_memory()
    layer.forward_infer_host(xh, yh, lh)
    np.testing.assert_array_equal(lh.numpy(), leaf_ref)
    util.check_outputs(yh, y_ref, cfg.dtype)
    layer.close()


@pytest.mark.parametrize("B", [16384, 40001])
def test_host_buffer_entry_point_chunked(B):
    """Batches of 16384 tokens or more go through the host entry point in overlapping chunks."""
    cfg = wl.FFFConfig("bf16_host_chunks", 128, 144, 4, 16, "gelu", "bf16", B, "normal")
    case = util.make_case(cfg, seed=3)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    layer = util.make_layer(case)
    xh = torch.from_numpy(case.x).to(torch.bfloat16).pin_memory()
    yh = torch.empty((B, cfg.O), dtype=torch.bfloat16).pin_memory()
    lh = torch.empty((B,), dtype=torch.int32).pin_memory()
    for _ in range(2):                                   # the second call reuses streams, events and staging
        yh.zero_()
        lh.fill_(-1)
        layer.forward_infer_host(xh, yh, lh)
        np.testing.assert_array_equal(lh.numpy(), leaf_ref)
        util.check_outputs(yh, y_ref, cfg.dtype)
    # the same rows through the device entry point, unchunked: identical bits (a row's result depends on no other row)
    y_dev, leaf_dev = layer.forward_infer(xh.cuda())
    torch.cuda.synchronize()
    assert torch.equal(y_dev.cpu(), yh)
    layer.close()


def test_gpu_argument_errors_are_reported_not_faulted():
    from paper_2308_14711_b200 import binding
    cfg = wl.FFFConfig("e", 16, 8, 2, 4, "relu", "f32", 8)
    case = util.Case(cfg, wl.make_weights(cfg, 0), None, None, 0)
    layer = util.make_layer(case)
    x = torch.zeros((8, 16), device="cuda")
    y = torch.zeros((8, 8), device="cuda")
    L = binding.lib()
    h = layer.handle
    assert L.fff_forward_infer(h, None, y.data_ptr(), None, 8, None) == 1
    assert L.fff_forward_infer(h, x.data_ptr(), None, None, 8, None) == 1
    assert L.fff_forward_infer(h, x.data_ptr() + 4, y.data_ptr(), None, 7, None) == 1     # misaligned
    assert L.fff_forward_infer(h, x.data_ptr(), y.data_ptr(), None, -1, None) == 1
    assert L.fff_forward_infer(h, x.data_ptr(), y.data_ptr(), None, 0, None) == 0         # empty batch
    assert L.fff_set_path(h, 9) == 1
    layer.close()
    assert L.fff_forward_infer(h, x.data_ptr(), y.data_ptr(), None, 8, None) == 6         # destroyed
    torch.cuda.synchronize()


@pytest.mark.parametrize("B,depth,l,x_kind", [(3000, 6, 32, "normal"), (1200, 6, 12, "normal"), (9000, 7, 64, "normal"),
                                              (6000, 7, 16, "clusters"), (700, 5, 24, "normal")])
def test_thin_buckets_on_the_tensor_core_leaf_kernel(B, depth, l, x_kind):
    """Buckets of a few dozen tokens: tiles of at most 32 / 64 rows are stacked four / two times in the rows of the
    second GEMM and every epilogue warp stores a share of their columns.  Results against the oracle, and bit for
    bit the same as the mma.sync kernel's routing and a second call (the scheduler words rearm themselves).
    The clustered inputs give buckets of several tiles next to empty ones; O = 272 ends in a 16-column piece."""
    cfg = wl.FFFConfig("bf16_thin", 256, 272, depth, l, "gelu" if l != 12 else "relu", "bf16", B, x_kind)
    case = util.make_case(cfg, seed=5)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    counts = np.bincount(leaf_ref, minlength=cfg.n_leaves)
    assert ((counts > 0) & (counts <= 32)).any() or ((counts > 32) & (counts <= 64)).any()
    layer = util.make_layer(case, "tensor")
    x = util.to_device(case.x, "bf16")
    y_first = None
    for _ in range(2):
        y, leaf = layer.forward_infer(x)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
        util.check_outputs(y, y_ref, "bf16")
        assert y_first is None or torch.equal(y, y_first)
        y_first = y.clone()
        assert layer.last_status() == 0
    layer.close()


def test_nonfinite_leaf_weights_stay_in_their_leaf():
    """Infinite output weights in one leaf make that leaf's tokens non-finite and leave every other token's
    result as the oracle has it (a tile holds one leaf's tokens only)."""
    cfg = wl.FFFConfig("bf16_inf_leaf", 128, 144, 5, 16, "gelu", "bf16", 1500, "normal")
    case = util.make_case(cfg, seed=2)
    bad = int(np.bincount(orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)[1], minlength=32).argmax())
    case.weights["w2"][bad, :, :] = np.inf
    case.net = orc.Net.from_config(cfg, case.weights)
    with np.errstate(all="ignore"):
        y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    layer = util.make_layer(case)
    y, leaf = layer.forward_infer(util.to_device(case.x, "bf16"))
    torch.cuda.synchronize()
    np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
    hit = leaf_ref == bad
    assert hit.any() and not hit.all()
    assert not np.isfinite(y_ref[hit]).all(axis=1).any()
    assert not torch.isfinite(y[torch.from_numpy(hit).cuda()].float()).all(dim=1).any()
    rows = np.nonzero(~hit)[0]
    util.check_outputs(y, y_ref[rows], "bf16", rows=rows)
    layer.close()


def test_descent_alone_then_forward():
    """The stage entry point for the descent, then whole forwards on the same handle: scratch that the descent
    leaves for the bucketing kernel must not leak from one call into the next."""
    cfg = wl.FFFConfig("bf16_d8_mixed_calls", 256, 64, 8, 8, "gelu", "bf16", 5000, "layernorm")
    case = util.make_case(cfg, seed=4)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    off_ref, perm_ref = orc.bucket(leaf_ref, cfg.n_leaves)
    layer = util.make_layer(case)
    x = util.to_device(case.x, "bf16")
    for _ in range(2):
        np.testing.assert_array_equal(layer.tree_descent(x).cpu().numpy(), leaf_ref)
        for _ in range(2):
            y, leaf = layer.forward_infer(x)
            torch.cuda.synchronize()
            np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
            off, perm = layer.last_bucketing(cfg.B)
            np.testing.assert_array_equal(off.cpu().numpy(), off_ref)
            np.testing.assert_array_equal(perm.cpu().numpy(), perm_ref)
            util.check_outputs(y, y_ref, "bf16")
    # a smaller batch afterwards: fewer tiles and blocks than the table has seen
    small = 700
    y, leaf = layer.forward_infer(x[:small])
    torch.cuda.synchronize()
    np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref[:small])
    off, perm = layer.last_bucketing(small)
    off_s, perm_s = orc.bucket(leaf_ref[:small], cfg.n_leaves)
    np.testing.assert_array_equal(off.cpu().numpy(), off_s)
    np.testing.assert_array_equal(perm.cpu().numpy(), perm_s)
    util.check_outputs(y, y_ref[:small], "bf16")
    assert layer.last_status() == 0
    layer.close()


@pytest.mark.parametrize("routing", ["spread", "one_leaf"])
def test_forward_without_bucketing_kernel(routing):
    """A tree of at most eight levels in front of the tensor-core leaf kernel: the descent files the tokens under
    their leaves itself, so a forward is two launches.  With zero node weights every logit is 0, which goes right
    (Algorithm 1: c >= 1/2), and the last leaf receives the whole batch: one list of many tiles, all others empty.
    The stable bucketing is still reported afterwards, and repeated calls start from cleared lists."""
    cfg = wl.FFFConfig("bf16_d5_direct", 256, 128, 5, 16, "gelu", "bf16", 3000, "normal")
    weights = wl.make_weights(cfg, 6)
    if routing == "one_leaf":
        weights["node_w"] = np.zeros_like(weights["node_w"])
        weights["node_b"] = np.zeros_like(weights["node_b"])
    net = orc.Net.from_config(cfg, weights)
    src = wl.TokenSource(cfg, 6)
    if routing == "spread":
        wl.enforce_margin(src, lambda rows: orc.path_margin(net, rows, threads=util.ORACLE_THREADS))
    case = util.Case(cfg, weights, net, src.x, 0)
    y_ref, leaf_ref = orc.forward_i(net, case.x, threads=util.ORACLE_THREADS)
    if routing == "one_leaf":
        assert (leaf_ref == cfg.n_leaves - 1).all()
    off_ref, perm_ref = orc.bucket(leaf_ref, cfg.n_leaves)
    layer = util.make_layer(case)
    x = util.to_device(case.x, "bf16")
    for B in (cfg.B, 1000, cfg.B):
        y, leaf = layer.forward_infer(x[:B])
        torch.cuda.synchronize()
        assert layer.last_launch_count() == 2
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref[:B])
        util.check_outputs(y, y_ref[:B], "bf16")
        off, perm = layer.last_bucketing(B)
        off_b, perm_b = (off_ref, perm_ref) if B == cfg.B else orc.bucket(leaf_ref[:B], cfg.n_leaves)
        np.testing.assert_array_equal(off.cpu().numpy(), off_b)
        np.testing.assert_array_equal(perm.cpu().numpy(), perm_b)
    assert layer.last_status() == 0
    layer.close()


@pytest.mark.parametrize("path,launches", [("warp", 3), ("auto", 1)])
@pytest.mark.parametrize("routing", ["spread", "one_leaf"])
def test_warp_kernels_changing_batch_sizes(routing, path, launches):
    """float32 layer with eight leaves, on the warp kernels (descent, bucketing, leaf: three launches) and on the default
    path (the one-launch kernel), also with every token in the last leaf (zero node weights: a logit of 0 goes right:
    one group of hidden neurons gets every token), and with batch sizes that change from call to call."""
    cfg = wl.FFFConfig("f32_d3_batches", 784, 10, 3, 32, "relu", "f32", 2048, "normal")
    weights = wl.make_weights(cfg, 3)
    if routing == "one_leaf":
        weights["node_w"] = np.zeros_like(weights["node_w"])
        weights["node_b"] = np.zeros_like(weights["node_b"])
    net = orc.Net.from_config(cfg, weights)
    src = wl.TokenSource(cfg, 3)
    if routing == "spread":
        wl.enforce_margin(src, lambda rows: orc.path_margin(net, rows, threads=util.ORACLE_THREADS))
    case = util.Case(cfg, weights, net, src.x, 0)
    y_ref, leaf_ref = orc.forward_i(net, case.x, threads=util.ORACLE_THREADS)
    if routing == "one_leaf":
        assert (leaf_ref == cfg.n_leaves - 1).all()
    layer = util.make_layer(case, path)
    x = util.to_device(case.x, "f32")
    for B in (cfg.B, 33, 1500, cfg.B):
        y, leaf = layer.forward_infer(x[:B])
        torch.cuda.synchronize()
        assert layer.last_launch_count() == launches
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref[:B])
        util.check_outputs(y, y_ref[:B], "f32")
        off, perm = layer.last_bucketing(B)
        off_b, perm_b = orc.bucket(leaf_ref[:B], cfg.n_leaves)
        np.testing.assert_array_equal(off.cpu().numpy(), off_b)
        np.testing.assert_array_equal(perm.cpu().numpy(), perm_b)
    assert layer.last_status() == 0
    layer.close()


def test_two_stage_descent_without_leaf_bucketing_kernel():
    """Ten levels as two tensor-core stages in front of the tensor-core leaf kernel: the first stage files the tokens
    under the nodes it reaches, the second derives its tiles from those lists and files the tokens under their leaves:
    three launches, no bucketing kernel at all.  The descent entry point alone is two launches and must leave nothing
    behind for the next forward.  With the direct lists switched off the two bucketing kernels are back."""
    cfg = wl.FFFConfig("bf16_d10_direct", 128, 64, 10, 16, "gelu", "bf16", 20000, "clusters")
    case = util.make_case(cfg, seed=8)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    layer = util.make_layer(case)
    x = util.to_device(case.x, "bf16")
    for B in (cfg.B, 17000, cfg.B):
        y, leaf = layer.forward_infer(x[:B])
        torch.cuda.synchronize()
        assert layer.last_launch_count() == 3
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref[:B])
        util.check_outputs(y, y_ref[:B], "bf16")
        off, perm = layer.last_bucketing(B)
        off_b, perm_b = orc.bucket(leaf_ref[:B], cfg.n_leaves)
        np.testing.assert_array_equal(off.cpu().numpy(), off_b)
        np.testing.assert_array_equal(perm.cpu().numpy(), perm_b)
        np.testing.assert_array_equal(layer.tree_descent(x[:B]).cpu().numpy(), leaf_ref[:B])
        assert layer.last_launch_count() == 2
    layer.set_tuning("direct_lists", False)
    y, leaf = layer.forward_infer(x)
    torch.cuda.synchronize()
    assert layer.last_launch_count() == 5          # stage, node bucketing, stage, leaf bucketing, leaf kernel
    np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
    util.check_outputs(y, y_ref, "bf16")
    assert layer.last_status() == 0
    layer.close()


def test_two_stage_descent_on_a_large_ragged_batch():
    """The node lists between the stages with many tiles per node, a ragged last tile in every list and skewed
    routing (some nodes empty, some with thousands of tokens): leaf indices bit-exact, outputs within tolerance."""
    for x_kind, B in (("normal", 200001), ("clusters", 150003)):
        cfg = wl.FFFConfig("bf16_d10_large", 128, 64, 10, 16, "relu", "bf16", B, x_kind)
        case = util.make_case(cfg, seed=12)
        y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
        layer = util.make_layer(case)
        y, leaf = layer.forward_infer(util.to_device(case.x, "bf16"))
        torch.cuda.synchronize()
        assert layer.last_launch_count() == 3 and layer.last_status() == 0
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
        util.check_outputs(y, y_ref, "bf16")
        layer.close()


def test_leaf_lists_too_large_fall_back_to_the_bucketing_kernel():
    """2048 leaves x 140 000 tokens x 4 bytes is more than the table of per-leaf lists may take (1 GiB): the forward
    then buckets by leaf with a kernel again (five launches) and reports that stable bucketing directly."""
    cfg = wl.FFFConfig("bf16_d11_big_batch", 128, 64, 11, 16, "gelu", "bf16", 140000, "normal")
    case = util.make_case(cfg, seed=11)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    off_ref, perm_ref = orc.bucket(leaf_ref, cfg.n_leaves)
    layer = util.make_layer(case)
    x = util.to_device(case.x, "bf16")
    for _ in range(2):
        y, leaf = layer.forward_infer(x)
        torch.cuda.synchronize()
        assert layer.last_launch_count() == 5
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
        util.check_outputs(y, y_ref, "bf16")
        off, perm = layer.last_bucketing(cfg.B)
        np.testing.assert_array_equal(off.cpu().numpy(), off_ref)
        np.testing.assert_array_equal(perm.cpu().numpy(), perm_ref)
    # a batch small enough for the lists on the same handle (the workspace keeps its size: still no lists)
    y, leaf = layer.forward_infer(x[:40000])
    torch.cuda.synchronize()
    np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref[:40000])
    util.check_outputs(y, y_ref[:40000], "bf16")
    assert layer.last_status() == 0
    layer.close()


@pytest.mark.parametrize("cfg", [
    wl.FFFConfig("graph_bf16_d6", 256, 128, 6, 16, "gelu", "bf16", 3000, "normal"),       # tensor kernels, direct leaf lists
    wl.FFFConfig("graph_bf16_d10", 128, 64, 10, 16, "gelu", "bf16", 20000, "clusters"),   # two descent stages, node bucketing
    wl.FFFConfig("graph_f32_d3", 784, 10, 3, 32, "relu", "f32", 517, "normal"),           # warp kernels
], ids=lambda c: c.name)
def test_forward_replayed_from_a_cuda_graph(cfg):
    """A forward enqueues kernels (and at most a small memset) on the caller's stream and, once the workspace has its
    size, neither allocates nor synchronises: it can be captured into a CUDA graph and replayed on new contents of
    the same buffers."""
    case = util.make_case(cfg, seed=9)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    layer = util.make_layer(case)
    layer.reserve(cfg.B)
    td = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    x_all = util.to_device(case.x, cfg.dtype)
    x = torch.zeros_like(x_all)
    y = torch.empty((cfg.B, cfg.O), dtype=td, device="cuda")
    leaf = torch.empty((cfg.B,), dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        layer.forward_infer(x, y=y, leaf_idx=leaf, stream=side)          # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        layer.forward_infer(x, y=y, leaf_idx=leaf, stream=torch.cuda.current_stream())
    for _ in range(2):
        y.zero_()
        leaf.fill_(-1)
        x.copy_(x_all)
        graph.replay()
        torch.cuda.synchronize()
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
        util.check_outputs(y, y_ref, cfg.dtype)
    assert layer.last_status() == 0
    del graph
    layer.close()


def test_nan_inputs_stay_in_range():
    cfg = wl.FFFConfig("n", 64, 32, 4, 8, "gelu", "bf16", 64)
    case = util.make_case(cfg, 0)
    layer = util.make_layer(case)
    x = util.to_device(case.x, "bf16")
    x[::3] = float("nan")
    y, leaf = layer.forward_infer(x)
    torch.cuda.synchronize()
    lf = leaf.cpu().numpy()
    assert ((lf >= 0) & (lf < 16)).all()
    assert torch.isnan(y[::3].float()).all()
    assert torch.isfinite(y[1::3].float()).all()
    layer.close()


@pytest.mark.parametrize("switch", ["tcgen05_descent", "tcgen05_grouped", "tcgen05_leaf", "cta_pairs", "direct_lists"])
def test_every_tuning_switch_off_gives_the_same_results(switch):
    """fff_set_tuning only chooses between kernels: with any one switch off, leaf indices and the bucketing stay
    bit-exact against the oracle and y within tolerance, on a two-stage tree (ten levels) and on a one-stage
    tree with more 128-token tiles than SMs (seven levels; the shape the CTA pairs serve)."""
    for cfg, seed in ((wl.FFFConfig("tune_d10", 128, 64, 10, 16, "gelu", "bf16", 20000, "clusters"), 8),
                      (wl.FFFConfig("tune_d7", 128, 64, 7, 8, "relu", "bf16", 20001, "normal"), 3)):
        case = util.make_case(cfg, seed=seed)
        y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
        off_ref, perm_ref = orc.bucket(leaf_ref, cfg.n_leaves)
        layer = util.make_layer(case)
        x = util.to_device(case.x, "bf16")
        y_on, _ = layer.forward_infer(x)
        launches_on = layer.last_launch_count()
        layer.set_tuning(switch, False)
        y, leaf = layer.forward_infer(x)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref)
        util.check_outputs(y, y_ref, "bf16")
        off, perm = layer.last_bucketing(cfg.B)
        np.testing.assert_array_equal(off.cpu().numpy(), off_ref)
        np.testing.assert_array_equal(perm.cpu().numpy(), perm_ref)
        if switch == "direct_lists":
            # the leaf bucketing kernel is back, and between two descent stages the node bucketing too
            assert layer.last_launch_count() == launches_on + (2 if cfg.depth > 8 else 1)
        layer.set_tuning(switch, True)
        y_back, _ = layer.forward_infer(x)
        assert torch.equal(y_back, y_on)
        assert layer.last_status() == 0
        layer.close()


@pytest.mark.parametrize("D", [256, 784])
@pytest.mark.parametrize("width,l", [(16, 1), (16, 8), (32, 2), (64, 4), (128, 1), (128, 8), (64, 1), (128, 2)])
def test_one_launch_kernel_on_the_shapes_of_the_papers_timing_tables(D, width, l):
    """float32 layers of the shape grid of Table 1 and the appendix table of inference times (inputs of 256 or 784,
    10 outputs, training width 16 to 128, leaves of 1 to 8 neurons, 2048 tokens): the default path is the
    one-launch kernel (several leaves share a group of 32 hidden neurons), checked against the oracle element by
    element, with the bucketing made on demand, twice in a row and on a shorter batch."""
    depth = (width // l).bit_length() - 1
    cfg = wl.FFFConfig(f"table1_D{D}_w{width}_l{l}", D, 10, depth, l, "relu", "f32", 2048, "normal", node_bias_std=0.1)
    case = util.make_case(cfg, seed=width + l)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    layer = util.make_layer(case)
    x = util.to_device(case.x, "f32")
    for B in (cfg.B, cfg.B, 777):
        y, leaf = layer.forward_infer(x[:B])
        torch.cuda.synchronize()
        assert layer.last_launch_count() == 1
        np.testing.assert_array_equal(leaf.cpu().numpy(), leaf_ref[:B])
        util.check_outputs(y, y_ref[:B], "f32")
        off, perm = layer.last_bucketing(B)
        off_b, perm_b = orc.bucket(leaf_ref[:B], cfg.n_leaves)
        np.testing.assert_array_equal(off.cpu().numpy(), off_b)
        np.testing.assert_array_equal(perm.cpu().numpy(), perm_b)
    # the three-kernel path gives the same leaves and outputs within the same tolerance
    layer.set_tuning("fused_small", False)
    y3, leaf3 = layer.forward_infer(x)
    torch.cuda.synchronize()
    assert layer.last_launch_count() > 1
    np.testing.assert_array_equal(leaf3.cpu().numpy(), leaf_ref)
    util.check_outputs(y3, y_ref, "f32")
    assert layer.last_status() == 0
    layer.close()


def test_a_bounded_wait_that_runs_out_is_reported_once_and_the_handle_stays_usable():
    """The error path of the tensor-core kernels' waits, exercised by the library's self-test kernel: a wait on a
    barrier that nothing signals gives up after 100 000 cycles (about 50 microseconds), the status word reports
    FFF_ERR_DEVICE_TIMEOUT exactly once, and forwards before and after it match the oracle."""
    from paper_2308_14711_b200 import binding
    cfg = wl.FFFConfig("timeout_probe", 128, 64, 5, 16, "gelu", "bf16", 1500, "normal")
    case = util.make_case(cfg, seed=4)
    y_ref, leaf_ref = orc.forward_i(case.net, case.x, threads=util.ORACLE_THREADS)
    layer = util.make_layer(case)
    x = util.to_device(case.x, "bf16")
    y, leaf = layer.forward_infer(x)
    assert layer.last_status() == 0
    binding.fff_selftest_bounded_wait(layer.handle, 100_000, torch.cuda.current_stream().cuda_stream)
    assert layer.last_status() == 5
    assert binding.status_string(5) == "device-side wait timed out"
    assert layer.last_status() == 0
    y2, leaf2 = layer.forward_infer(x)
    torch.cuda.synchronize()
    assert layer.last_status() == 0
    np.testing.assert_array_equal(leaf2.cpu().numpy(), leaf_ref)
    util.check_outputs(y2, y_ref, "bf16")
    assert torch.equal(y, y2)
    with pytest.raises(Exception):
        binding.fff_selftest_bounded_wait(layer.handle, 0)
    layer.close()


def test_capabilities_say_which_kernel_families_a_layer_can_use():
    def caps(D, O, depth, l, dtype):
        cfg = wl.FFFConfig("caps", D, O, depth, l, "relu", dtype, 4, "normal")
        layer = util.make_layer(util.make_case(cfg, seed=1, margin=None))
        c = layer.capabilities()
        layer.close()
        return c
    full = caps(256, 128, 4, 16, "bf16")
    assert full & 1 and full & 2 and full & 4 and full & 8 and full & 16 and full & 32
    assert not full & 64                               # grouped leaf tiles: thin leaves under deep trees only
    assert caps(256, 128, 9, 12, "bf16") & 64
    odd_d = caps(192, 128, 4, 16, "bf16")              # D no multiple of 128: CUDA cores only, FORWARD_T still runs
    assert not odd_d & (1 | 2 | 4 | 8) and odd_d & 16 and odd_d & 32
    odd_o = caps(256, 100, 4, 16, "bf16")              # O no multiple of 8: descent on tensor cores, leaves not
    assert odd_o & 1 and not odd_o & (4 | 8)
    f32 = caps(256, 128, 4, 16, "f32")
    assert f32 == 16
    wide = caps(256, 128, 2, 48, "f32")                # leaves wider than 32: no one-launch kernel
    assert wide == 0
