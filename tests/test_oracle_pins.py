"""Pins of the CPU oracle against facts it does not compute itself.

Each test checks the oracle against something fixed by the paper or by
mathematics: brute-force region membership, hand-computed values, library
routines (torch / numpy), identities stated in the paper, printed table values.
"""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import fff_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_net(rng, D, O, depth, l, act, node_bias=True, scale=1.0):
    nn, nl = (1 << depth) - 1, 1 << depth
    return orc.Net(D, O, depth, l, act,
                   rng.standard_normal((nn, D)) * scale,
                   rng.standard_normal(nn) * (scale if node_bias else 0.0),
                   rng.standard_normal((nl, l, D)) / math.sqrt(D),
                   rng.standard_normal((nl, l)) * 0.3,
                   rng.standard_normal((nl, O, l)) / math.sqrt(l),
                   rng.standard_normal((nl, O)) * 0.3)


# ---------------------------------------------------------------- routing rule
@pytest.mark.parametrize("depth", [1, 2, 3, 4])
def test_descent_matches_brute_force_region_membership(depth):
    """Algorithm 1: exactly one leaf's root path accepts each input, and it is the one reached."""
    rng = np.random.default_rng(depth)
    net = rand_net(rng, 5, 3, depth, 2, "relu")
    x = rng.standard_normal((200, 5))
    leaf, _, _ = orc.descend(net, x)
    for t in range(x.shape[0]):
        hits, j = orc.brute_force_leaf(net, x[t])
        assert hits == 1
        assert j == leaf[t]
    assert len(set(leaf.tolist())) > 1


def test_hand_computed_descent_and_leaf_values():
    """d=2, D=2, l=2, O=3 with small integers; every number below was worked out by hand."""
    # nodes (breadth-first): N00: x0 - x1 + 0.5 ; N10: x0 + x1 - 1 ; N11: -x0 + 2
    node_w = [[1, -1], [1, 1], [-1, 0]]
    node_b = [0.5, -1, 2]
    # leaf j: W1 = [[j+1, 0], [0, -(j+1)]], b1 = [0, 1]; W2 = [[1, 0], [0, 1], [1, 1]], b2 = [j, 0, -1]
    w1 = [[[j + 1, 0], [0, -(j + 1)]] for j in range(4)]
    b1 = [[0, 1]] * 4
    w2 = [[[1, 0], [0, 1], [1, 1]]] * 4
    b2 = [[j, 0, -1] for j in range(4)]
    net = orc.Net(2, 3, 2, 2, "relu", node_w, node_b, w1, b1, w2, b2)
    x = np.array([
        [2.0, 0.0],    # N00: 2.5>=0 right -> N11: 0>=0 right (tie) -> leaf 3
        [0.0, 2.0],    # N00: -1.5 left -> N10: 1>=0 right -> leaf 1
        [0.0, 0.75],   # N00: -0.25 left -> N10: -0.25 left -> leaf 0
        [3.0, 1.0],    # N00: 2.5 right -> N11: -1 left -> leaf 2
        [-1.0, -0.5],  # N00: 0.0>=0 right (tie) -> N11: 3 right -> leaf 3
    ])
    y, leaf = orc.forward_i(net, x)
    assert leaf.tolist() == [3, 1, 0, 2, 3]
    # leaf 3 on (2,0): h = relu([8, 1]) = [8,1]; y = [8+3, 1, 9-1]
    # leaf 1 on (0,2): h = relu([0, -4+1]) = [0,0]; y = [1, 0, -1]
    # leaf 0 on (0,.75): h = relu([0, -.75+1]) = [0,.25]; y = [0, .25, -.75]
    # leaf 2 on (3,1): h = relu([9, -3+1]) = [9,0]; y = [9+2, 0, 8]
    # leaf 3 on (-1,-.5): h = relu([-4, 2+1]) = [0,3]; y = [3, 3, 2]
    expect = np.array([[11, 1, 8], [1, 0, -1], [0, 0.25, -0.75], [11, 0, 8], [3, 3, 2]], float)
    np.testing.assert_allclose(y, expect, rtol=0, atol=1e-15)
    # smallest |logit| on each token's path, from the logits worked out above:
    # (2.5, 0) -> 0; (-1.5, 1) -> 1; (-0.25, -0.25) -> 0.25; (2.5, -1) -> 1; (0, 3) -> 0
    leaf_d, margin, _ = orc.descend(net, x)
    assert leaf_d.tolist() == [3, 1, 0, 2, 3]
    assert margin.tolist() == [0.0, 1.0, 0.25, 1.0, 0.0]
    assert orc.path_margin(net, x).tolist() == [0.0, 1.0, 0.25, 1.0, 0.0]


def test_tie_goes_right_zero_node_weights_reach_last_leaf():
    """c = 1/2 satisfies c >= 1/2, so with all node weights zero every token ends in leaf 2^d - 1."""
    rng = np.random.default_rng(0)
    for depth in (1, 3, 5):
        net = rand_net(rng, 4, 2, depth, 2, "gelu")
        net.node_w[:] = 0.0
        net.node_b[:] = 0.0
        leaf, mn, _ = orc.descend(net, rng.standard_normal((17, 4)))
        assert (leaf == (1 << depth) - 1).all()
        assert (mn == 0).all()
        net.node_b[:] = -0.0          # negative zero is still >= 0
        assert (orc.descend(net, rng.standard_normal((3, 4)))[0] == (1 << depth) - 1).all()


def test_exactly_d_nodes_and_one_leaf_per_token():
    rng = np.random.default_rng(1)
    for depth in (0, 1, 4):
        net = rand_net(rng, 6, 3, depth, 2, "relu")
        counters = {}
        orc.forward_i(net, rng.standard_normal((37, 6)), counters=counters)
        assert counters["node_evals"] == 37 * depth
        assert counters["leaf_evals"] == 37


# ---------------------------------------------------------------- leaf evaluation
@pytest.mark.parametrize("act", ["relu", "gelu", "gelu_tanh", "silu"])
def test_depth_zero_is_a_plain_feedforward_layer(act):
    """d = 0: no nodes, one leaf -- the network is an ordinary <D, l, O> layer (library ops)."""
    rng = np.random.default_rng(2)
    D, l, O = 11, 7, 5
    net = rand_net(rng, D, O, 0, l, act)
    x = rng.standard_normal((23, D))
    y, leaf = orc.forward_i(net, x)
    assert (leaf == 0).all()
    xt = torch.from_numpy(x)
    h = F.linear(xt, torch.from_numpy(net.w1[0]), torch.from_numpy(net.b1[0]))
    # torch's default GELU is the exact erf form
    h = {"relu": F.relu, "gelu": F.gelu, "gelu_tanh": lambda v: F.gelu(v, approximate="tanh"), "silu": F.silu}[act](h)
    ref = F.linear(h, torch.from_numpy(net.w2[0]), torch.from_numpy(net.b2[0])).numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-13)


def test_gelu_known_values():
    """GELU(v) = v Phi(v): Phi(1), Phi(2) from standard normal tables; GELU(-v) = GELU(v) - v."""
    # D=1, l=1, O=1, W1=1, b1=0, W2=1, b2=0  => y = GELU(x)
    net = orc.Net(1, 1, 0, 1, "gelu", None, None, [[[1.0]]], [[0.0]], [[[1.0]]], [[0.0]])
    x = np.array([[0.0], [1.0], [2.0], [-1.0], [30.0], [-30.0]])
    y, _ = orc.forward_i(net, x)
    phi1, phi2 = 0.8413447460685429, 0.9772498680518208
    np.testing.assert_allclose(y[:, 0], [0.0, phi1, 2 * phi2, phi1 - 1.0, 30.0, 0.0], rtol=0, atol=1e-15)


@pytest.mark.parametrize("act", ["gelu_tanh", "silu"])
def test_smooth_activations_known_values_and_identity(act):
    """Both are v times an increasing function s with s(v) + s(-v) = 1, so f(v) - f(-v) = v, f(0) = 0, f(v) -> v and
    f(-v) -> 0 far from zero; SiLU(1) = 1 / (1 + e^-1); tanh-GELU(1) = (1 + tanh(sqrt(2/pi) * 1.044715)) / 2; and the
    tanh form stays within 5e-4 of the exact GELU everywhere, yet is not equal to it."""
    net = orc.Net(1, 1, 0, 1, act, None, None, [[[1.0]]], [[0.0]], [[[1.0]]], [[0.0]])
    v = np.array([0.0, 1.0, -1.0, 2.5, -2.5, 40.0, -40.0, 0.3, -0.3])
    y = orc.forward_i(net, v[:, None])[0][:, 0]
    assert y[0] == 0.0
    np.testing.assert_allclose(y[1::2] - y[2::2], v[1::2], rtol=0, atol=1e-14)
    np.testing.assert_allclose(y[5:7], [40.0, 0.0], rtol=0, atol=1e-15)
    one = 1.0 / (1.0 + np.exp(-1.0)) if act == "silu" else 0.5 * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * 1.044715))
    np.testing.assert_allclose(y[1], one, rtol=1e-15)
    if act == "gelu_tanh":
        exact = orc.Net(1, 1, 0, 1, "gelu", None, None, [[[1.0]]], [[0.0]], [[[1.0]]], [[0.0]])
        grid = np.linspace(-6, 6, 2401)[:, None]
        diff = np.abs(orc.forward_i(net, grid)[0] - orc.forward_i(exact, grid)[0])
        assert 1e-5 < diff.max() < 5e-4


def test_leaf_biases_and_w2_orientation_matter():
    """O != l and non-zero biases: a transposed W2 or a dropped bias changes this hand case."""
    # D=1, l=2, O=3: h = relu([x+1, -x]) ; y = W2 h + b2
    net = orc.Net(1, 3, 0, 2, "relu", None, None, [[[1.0], [-1.0]]], [[1.0, 0.0]],
                  [[[1.0, 2.0], [3.0, 4.0], [5.0, 6.0]]], [[0.5, -0.5, 0.25]])
    y, _ = orc.forward_i(net, np.array([[2.0], [-3.0]]))
    # x=2: h=[3,0] -> [3.5, 8.5, 15.25];  x=-3: h=[0,3] -> [6.5, 11.5, 18.25]
    np.testing.assert_allclose(y, [[3.5, 8.5, 15.25], [6.5, 11.5, 18.25]], rtol=0, atol=1e-15)


# ---------------------------------------------------------------- hard vs soft
def test_soft_mixture_with_zero_nodes_is_mean_of_leaves_as_wide_layer():
    """All node weights 0 => every c = 1/2 => FORWARD_T is a width 2^d*l layer with output weights / 2^d."""
    rng = np.random.default_rng(3)
    D, O, depth, l = 6, 4, 3, 5
    net = rand_net(rng, D, O, depth, l, "gelu")
    net.node_w[:] = 0.0
    net.node_b[:] = 0.0
    x = rng.standard_normal((9, D))
    y = orc.forward_t(net, x)
    nl = 1 << depth
    W1 = torch.from_numpy(net.w1.reshape(nl * l, D))
    B1 = torch.from_numpy(net.b1.reshape(nl * l))
    W2 = torch.from_numpy(np.concatenate([net.w2[j] for j in range(nl)], axis=1) / nl)   # [O, nl*l]
    B2 = torch.from_numpy(net.b2.mean(axis=0))
    ref = F.linear(F.gelu(F.linear(torch.from_numpy(x), W1, B1)), W2, B2).numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-13)


def test_soft_mixture_weights_sum_to_one():
    """Leaves that all output the constant 1 make FORWARD_T return the sum of the choice vector c."""
    rng = np.random.default_rng(4)
    net = rand_net(rng, 5, 2, 4, 3, "relu")
    net.w2[:] = 0.0
    net.b2[:] = 1.0
    y = orc.forward_t(net, rng.standard_normal((11, 5)))
    np.testing.assert_allclose(y, 1.0, rtol=0, atol=1e-14)


def test_soft_mixture_follows_the_choice_product_on_a_depth_one_tree():
    """d = 1: FORWARD_T = c * right leaf + (1 - c) * left leaf with c = sigmoid(logit), by hand."""
    # node: logit = 2x ; leaves (D=1,l=1,O=1, relu): left y = relu(x) * 1 + 10 ; right y = relu(x) * 3 - 10
    net = orc.Net(1, 1, 1, 1, "relu", [[2.0]], [0.0], [[[1.0]], [[1.0]]], [[0.0], [0.0]],
                  [[[1.0]], [[3.0]]], [[10.0], [-10.0]])
    x = np.array([[0.5], [-1.0]])
    y = orc.forward_t(net, x)
    c = [1 / (1 + math.exp(-1.0)), 1 / (1 + math.exp(2.0))]
    expect = [c[0] * (1.5 - 10) + (1 - c[0]) * (0.5 + 10), c[1] * (-10.0) + (1 - c[1]) * 10.0]
    np.testing.assert_allclose(y[:, 0], expect, rtol=1e-15)


@pytest.mark.parametrize("act", ["relu", "gelu", "gelu_tanh", "silu"])
def test_hard_inference_is_the_saturated_limit_of_the_soft_mixture(act):
    """Rescaling node coefficients squashes the sigmoid to a step: FORWARD_T -> FORWARD_I."""
    rng = np.random.default_rng(5)
    D, O, depth, l = 8, 3, 4, 3
    net = rand_net(rng, D, O, depth, l, act)
    x = rng.standard_normal((64, D))
    _, mn, _ = orc.descend(net, x)
    x = x[mn >= 1e-2]
    assert x.shape[0] > 40
    y_hard, _ = orc.forward_i(net, x)
    hard = orc.Net(D, O, depth, l, act, net.node_w * 1e4, net.node_b * 1e4, net.w1, net.b1, net.w2, net.b2)
    np.testing.assert_array_equal(orc.descend(hard, x)[0], orc.descend(net, x)[0])
    np.testing.assert_allclose(orc.forward_t(hard, x), y_hard, rtol=1e-12, atol=1e-12)


def test_conditional_execution_equals_all_leaves_masked():
    rng = np.random.default_rng(6)
    net = rand_net(rng, 7, 4, 3, 3, "gelu")
    x = rng.standard_normal((50, 7))
    y, leaf = orc.forward_i(net, x)
    np.testing.assert_allclose(orc.forward_all_leaves_masked(net, x, leaf), y, rtol=1e-14, atol=1e-14)
    wrong = (leaf + 1) % 8
    assert np.abs(orc.forward_all_leaves_masked(net, x, wrong) - y).max() > 1e-3


def test_threads_do_not_change_results():
    rng = np.random.default_rng(7)
    net = rand_net(rng, 9, 4, 3, 3, "gelu")
    x = rng.standard_normal((101, 9))
    y1, l1 = orc.forward_i(net, x, threads=1)
    y4, l4 = orc.forward_i(net, x, threads=4)
    np.testing.assert_array_equal(y1, y4)
    np.testing.assert_array_equal(l1, l4)


# ---------------------------------------------------------------- sizes
def test_sizes_match_table_3():
    rows = [list(map(int, ln.split())) for ln in open(os.path.join(GOLDEN, "table3_sizes.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 6
    for l, d, tw, ts, iw, isz in rows:
        assert orc.training_width(d, l) == tw
        assert orc.training_size(d, 1, l) == ts
        assert orc.inference_width(l) == iw
        assert orc.inference_size(d, 1, l) == isz


# ---------------------------------------------------------------- bucketing
@pytest.mark.parametrize("B,nl", [(0, 4), (1, 1), (257, 8), (1000, 64), (5000, 3)])
def test_bucketing_is_the_stable_sort_by_leaf(B, nl):
    rng = np.random.default_rng(B + nl)
    leaf = rng.integers(0, nl, size=B).astype(np.int32)
    if B > 10:
        leaf[: B // 2] = leaf[0]          # a heavy bucket
    offsets, perm = orc.bucket(leaf, nl)
    assert offsets[0] == 0 and offsets[-1] == B
    np.testing.assert_array_equal(np.diff(offsets), np.bincount(leaf, minlength=nl))
    np.testing.assert_array_equal(perm, np.argsort(leaf, kind="stable"))
    assert sorted(perm.tolist()) == list(range(B))
    for j in range(nl):
        seg = perm[offsets[j]:offsets[j + 1]]
        assert (leaf[seg] == j).all()
        assert (np.diff(seg) > 0).all()


def test_mean_bucket_size_is_batch_over_leaves():
    """Batch 256 over 128 leaves: 2 samples per leaf on average (explorative evaluation, l=1, w=128)."""
    leaf = np.random.default_rng(0).integers(0, 128, size=256).astype(np.int32)
    offsets, _ = orc.bucket(leaf, 128)
    assert np.diff(offsets).mean() == 2.0


# ---- the stack oracle (several FFF blocks with layer normalisation and residual connections) ----------------

def test_stack_layer_norm_is_the_library_layer_norm():
    from oracle import fff_stack_oracle as so
    rng = np.random.default_rng(7)
    x = rng.standard_normal((9, 33)) * 3.0 + 1.5
    g, b = rng.standard_normal(33), rng.standard_normal(33)
    ref = F.layer_norm(torch.from_numpy(x), (33,), torch.from_numpy(g), torch.from_numpy(b), eps=1e-5).numpy()
    np.testing.assert_allclose(so.layer_norm(x, g, b, 1e-5), ref, rtol=1e-12, atol=1e-13)
    plain = F.layer_norm(torch.from_numpy(x), (33,), eps=1e-3).numpy()
    np.testing.assert_allclose(so.layer_norm(x, None, None, 1e-3), plain, rtol=1e-12, atol=1e-13)


def test_stack_storage_rounding_is_the_library_conversion():
    from oracle import fff_stack_oracle as so
    rng = np.random.default_rng(8)
    a = np.concatenate([rng.standard_normal(4000) * 10.0 ** rng.integers(-6, 6, 4000), [0.0, -0.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8]])
    ref = torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16).double().numpy()
    np.testing.assert_array_equal(so.store(a, "bf16"), ref)
    np.testing.assert_array_equal(so.store(a, "f32"), a.astype(np.float32).astype(np.float64))


def test_stack_of_one_plain_block_is_forward_i_and_zero_leaves_make_the_identity():
    from oracle import fff_stack_oracle as so
    rng = np.random.default_rng(9)
    D = 12
    nets = [rand_net(rng, D, D, 3, 4, "gelu") for _ in range(3)]
    x = rng.standard_normal((40, D))
    y1, leaves, margin = so.stack_forward(nets[:1], x, "f32", norms=None, residual=False)
    y_ref, leaf_ref = orc.forward_i(nets[0], x)
    np.testing.assert_array_equal(leaves[0], leaf_ref)
    np.testing.assert_array_equal(y1, y_ref.astype(np.float32).astype(np.float64))
    np.testing.assert_array_equal(margin, orc.path_margin(nets[0], x))
    # residual blocks whose leaves output zero leave the token unchanged, whatever the normalisation does
    for n in nets:
        n.w2[:] = 0.0
        n.b2[:] = 0.0
    norms = [(rng.standard_normal(D), rng.standard_normal(D)), None, (None, None)]
    x32 = x.astype(np.float32).astype(np.float64)
    y3, leaves3, _ = so.stack_forward(nets, x32, "f32", norms=norms, residual=True)
    np.testing.assert_array_equal(y3, x32)
    assert len(leaves3) == 3
    # two blocks by hand: x1 = x0 + f0(LN(x0)), x2 = x1 + f1(x1)
    nets2 = [rand_net(rng, D, D, 2, 3, "relu") for _ in range(2)]
    z0 = so.layer_norm(x32, norms[0][0], norms[0][1], 1e-5).astype(np.float32).astype(np.float64)
    x1 = (x32 + orc.forward_i(nets2[0], z0)[0]).astype(np.float32).astype(np.float64)
    x2 = (x1 + orc.forward_i(nets2[1], x1)[0]).astype(np.float32).astype(np.float64)
    got, _, _ = so.stack_forward(nets2, x32, "f32", norms=[norms[0], None], residual=True)
    np.testing.assert_array_equal(got, x2)


# ---- FORWARD_T by products over paths, and node entropies --------------------------------------------------

def test_mixture_weights_are_stochastic_and_reproduce_the_recursive_forward_t():
    """The product form and the recursion of Algorithm 1 are two separate pieces of code: sum_j mix_j leaf_j(x)
    must equal FORWARD_T, each row of weights must sum to 1, and d = 1 is (1 - c, c) by hand."""
    rng = np.random.default_rng(11)
    for depth in (1, 2, 4):
        net = rand_net(rng, 5, 3, depth, 2, "gelu")
        x = rng.standard_normal((13, 5))
        mix = orc.mixture_weights(net, x, threads=2)
        assert mix.shape == (13, 1 << depth) and (mix >= 0).all()
        np.testing.assert_allclose(mix.sum(axis=1), 1.0, rtol=0, atol=1e-14)
        leaves = np.stack([orc.forward_all_leaves_masked(net, x, np.full(13, j, np.int32)) for j in range(1 << depth)], axis=1)
        np.testing.assert_allclose((mix[:, :, None] * leaves).sum(axis=1), orc.forward_t(net, x), rtol=1e-12, atol=1e-13)
        np.testing.assert_array_equal(orc.forward_t_rows(net, x, threads=3), orc.forward_t(net, x))
    net = rand_net(rng, 2, 1, 1, 1, "relu")
    net.node_w[:] = [[2.0, -1.0]]
    net.node_b[:] = [0.5]
    c = 1.0 / (1.0 + np.exp(-(2.0 * 0.25 - 1.0 * 3.0 + 0.5)))
    np.testing.assert_allclose(orc.mixture_weights(net, [[0.25, 3.0]]), [[1.0 - c, c]], rtol=1e-15)
    # on the path of the hard descent every factor is at least 1/2: that leaf's weight is at least 2^-d
    net = rand_net(rng, 6, 2, 3, 2, "relu")
    x = rng.standard_normal((50, 6))
    mix = orc.mixture_weights(net, x)
    assert (mix[np.arange(50), orc.descend(net, x)[0]] >= 0.125).all()


def test_node_entropy_closed_forms_and_library_routine():
    """c = 1/2 everywhere gives ln 2 per node; saturated nodes give 0; a hand case against scipy's entropy."""
    from scipy.stats import entropy
    rng = np.random.default_rng(12)
    net = rand_net(rng, 4, 2, 3, 2, "relu")
    x = rng.standard_normal((20, 4))
    keep_w, keep_b = net.node_w.copy(), net.node_b.copy()
    net.node_w[:] = 0.0
    net.node_b[:] = 0.0
    np.testing.assert_allclose(orc.node_entropy(net, x), np.log(2.0), rtol=1e-14)
    net.node_w[:] = keep_w * 1e4
    net.node_b[:] = keep_b * 1e4
    assert orc.node_entropy(net, x).max() < 1e-3          # one token may sit within 1e-4 of a boundary
    net.node_w[:], net.node_b[:] = keep_w, keep_b
    ent = orc.node_entropy(net, x)
    assert ent.shape == (7,) and (ent > 0).all() and (ent <= np.log(2.0)).all()
    for r in (0, 3, 6):                         # every node sees every token
        c = 1.0 / (1.0 + np.exp(-(x @ keep_w[r] + keep_b[r])))
        ref = np.mean([entropy([ci, 1.0 - ci]) for ci in c])
        np.testing.assert_allclose(ent[r], ref, rtol=1e-12)
