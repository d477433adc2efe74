"""GPU parity of stacks of FFF layers (layer normalisation, residual connections, CUDA-graph replay) against the
float64 stack oracle.

Tokens are independent through the whole stack, so the inputs are margin-enforced for ALL layers at once: a token
is redrawn until no routing logit of any layer, as the oracle computes them from its own intermediate values, is
within the margin of zero.  For float32 stacks that is the single-layer margin 1e-2.  In a bf16 stack the input
of a later layer already carries the earlier layers' bf16-level deviations (outputs within 2e-2 (1 + |ref|), in
practice a few 1e-3 per element, which a routing logit over D = 256 features with weights of variance 1/D turns into
deviations of about 5e-3), so the margin there is 5e-2, ten times that.  Leaf indices of every layer are then
bit-exact.  The final output of a float32 stack is held to the single-layer tolerance; that of a bf16 stack of K
blocks to K times the single-layer tolerance (|err| <= K 2e-2 (1 + |ref|), relative L2 <= K 1e-2): every block adds
a deviation within the single-layer tolerance and hands the earlier ones on through its residual connection.
"""
import numpy as np
import pytest
import torch

from oracle import fff_oracle as orc
from oracle import fff_stack_oracle as so
from paper_2308_14711_b200 import workloads as wl
from paper_2308_14711_b200.binding import FFFStack
from tests import util

pytestmark = pytest.mark.gpu

MARGIN = {"f32": wl.DEFAULT_MARGIN, "bf16": 5e-2}


def tol_scale(cfg, n_layers):
    return float(n_layers) if cfg.dtype == "bf16" else 1.0


def build(cfg, n_layers, seed, layer_norm, residual, affine=True):
    rng = np.random.default_rng(seed)
    weights = [wl.make_weights(cfg, seed + 17 * k) for k in range(n_layers)]
    nets = [orc.Net.from_config(cfg, w) for w in weights]
    if layer_norm:
        def vec(center):
            v = (center + 0.2 * rng.standard_normal(cfg.D)).astype(np.float32)
            return wl.round_to_bf16(v) if cfg.dtype == "bf16" else v
        norms = [(vec(1.0), vec(0.0)) if affine or k % 2 == 0 else (None, None) for k in range(n_layers)]
    else:
        norms = None
    src = wl.TokenSource(cfg, seed)
    wl.enforce_margin(src, lambda rows: so.stack_forward(nets, rows, cfg.dtype, norms, 1e-5, residual, threads=util.ORACLE_THREADS)[2],
                      margin=MARGIN[cfg.dtype])
    cases = [util.Case(cfg, w, n, None, 0) for w, n in zip(weights, nets)]
    return cases, nets, norms, src.x


def run(cfg, n_layers, seed, layer_norm, residual, affine=True, graph=False, path="auto"):
    cases, nets, norms, x_host = build(cfg, n_layers, seed, layer_norm, residual, affine)
    y_ref, leaves_ref, margin = so.stack_forward(nets, x_host, cfg.dtype, norms, 1e-5, residual, threads=util.ORACLE_THREADS)
    assert margin.min() >= MARGIN[cfg.dtype]
    layers = [util.make_layer(c, path) for c in cases]
    gam = bet = None
    if norms is not None:
        gam = [None if g is None else util.to_device(g, cfg.dtype) for g, _ in norms]
        bet = [None if b is None else util.to_device(b, cfg.dtype) for _, b in norms]
    stack = FFFStack(layers, layer_norm=layer_norm, gammas=gam, betas=bet, eps=1e-5, residual=residual)
    stack.set_graph(graph)
    x = util.to_device(x_host, cfg.dtype)
    y = torch.empty_like(x)
    leaf = torch.empty((n_layers, cfg.B), dtype=torch.int32, device="cuda")
    replays = 0
    # (a recording needs a stream of its own: the legacy default stream cannot be captured)
    side = torch.cuda.Stream() if graph else None
    torch.cuda.synchronize()
    for it in range(4 if graph else 2):
        y.fill_(7.0)
        torch.cuda.synchronize()
        stack.forward(x, y, leaf, stream=side)
        torch.cuda.synchronize()
        replays += stack.last_was_replay()
        for k in range(n_layers):
            np.testing.assert_array_equal(leaf[k].cpu().numpy(), leaves_ref[k], err_msg=f"layer {k}, call {it}")
        util.check_outputs(y, y_ref, cfg.dtype, scale=tol_scale(cfg, n_layers))
        for l in layers:
            assert l.last_status() == 0
    if graph:
        assert replays >= 2, "the third and fourth calls with the same arguments must be replays"
        # new contents at the recorded addresses are read by the replay
        x2_host = np.ascontiguousarray(x_host[::-1])
        y2_ref, leaves2_ref, _ = so.stack_forward(nets, x2_host, cfg.dtype, norms, 1e-5, residual, threads=util.ORACLE_THREADS)
        x.copy_(util.to_device(x2_host, cfg.dtype))
        torch.cuda.synchronize()
        stack.forward(x, y, leaf, stream=side)
        torch.cuda.synchronize()
        assert stack.last_was_replay()
        for k in range(n_layers):
            np.testing.assert_array_equal(leaf[k].cpu().numpy(), leaves2_ref[k])
        util.check_outputs(y, y2_ref, cfg.dtype, scale=tol_scale(cfg, n_layers))
        # other arguments: plain launches again
        y_other, _ = stack.forward(x[:100].contiguous(), stream=side)
        torch.cuda.synchronize()
        assert not stack.last_was_replay()
        util.check_outputs(y_other, y2_ref[:100], cfg.dtype, scale=tol_scale(cfg, n_layers))
    stack.close()
    for l in layers:
        l.close()


@pytest.mark.parametrize("layer_norm,residual,affine", [(True, True, True), (True, True, False), (False, True, True),
                                                        (True, False, True), (False, False, True)])
def test_float32_stack_matches_the_stack_oracle(layer_norm, residual, affine):
    cfg = wl.FFFConfig("stack_f32", 96, 96, 3, 8, "gelu", "f32", 700, "normal", node_bias_std=0.2)
    run(cfg, 3, 21, layer_norm, residual, affine)


@pytest.mark.parametrize("graph", [False, True])
def test_bf16_stack_on_the_tensor_core_kernels(graph):
    """Four layers of 256 features, 64 leaves of width 16 each (the tensor-core descent with direct leaf lists and
    the tensor-core leaf kernel), with layer normalisation and residual connections; plain launches and graph replay."""
    cfg = wl.FFFConfig("stack_bf16", 256, 256, 6, 16, "gelu", "bf16", 6000, "normal")
    run(cfg, 4, 5, True, True, graph=graph)


def test_float32_stack_replayed_from_a_graph():
    """The one-launch kernel of small float32 layers is a cooperative launch; the stack records it too, or falls
    back to plain launches: either way the results are the oracle's."""
    cfg = wl.FFFConfig("stack_f32_graph", 64, 64, 2, 16, "relu", "f32", 900, "normal", node_bias_std=0.3)
    cases, nets, norms, x_host = build(cfg, 2, 3, True, True)
    y_ref, leaves_ref, _ = so.stack_forward(nets, x_host, cfg.dtype, norms, 1e-5, True, threads=util.ORACLE_THREADS)
    layers = [util.make_layer(c) for c in cases]
    stack = FFFStack(layers, True, [util.to_device(g, "f32") for g, _ in norms], [util.to_device(b, "f32") for _, b in norms])
    stack.set_graph(True)
    x = util.to_device(x_host, "f32")
    y = torch.empty_like(x)
    leaf = torch.empty((2, cfg.B), dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(4):
        stack.forward(x, y, leaf, stream=side)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(leaf[1].cpu().numpy(), leaves_ref[1])
        util.check_outputs(y, y_ref, "f32")
    stack.close()
    for l in layers:
        l.close()


def test_stack_argument_errors():
    from paper_2308_14711_b200 import binding
    cfg_a = wl.FFFConfig("stack_a", 64, 64, 2, 8, "relu", "f32", 10, "normal")
    cfg_b = wl.FFFConfig("stack_b", 64, 32, 2, 8, "relu", "f32", 10, "normal")
    la = util.make_layer(util.make_case(cfg_a, 1))
    lb = util.make_layer(util.make_case(cfg_b, 1))
    with pytest.raises(binding.FFFError):
        FFFStack([la, lb])                  # widths differ
    with pytest.raises(binding.FFFError):
        FFFStack([la, la])                  # one handle twice
    assert binding.lib().fff_stack_destroy(None) == 6
    assert binding.lib().fff_stack_forward(None, None, None, None, 1, None) == 6
    s = FFFStack([la], layer_norm=False, residual=False)
    y, _ = s.forward(torch.zeros((0, 64), device="cuda"))
    assert y.shape == (0, 64)
    s.close()
    la.close()
    lb.close()
