"""Pins of the oracle's unmasked back-propagation helpers (the steps that chain
the masked products into a training step) against float64 autograd of the
library's own convolution, ReLU and max pooling on the CPU, and of the
aggregation over virtual batches against linearity."""
import numpy as np
import pytest
import torch
import torch.nn.functional as TF

from oracle import dk_oracle as O
from paper_2207_00083_b200 import synth


def t64(a, grad=False):
    return torch.tensor(np.asarray(a, dtype=np.float64), requires_grad=grad)


@pytest.mark.parametrize("k,s,p,h,w", [(3, 1, 1, 6, 5), (3, 2, 1, 7, 7), (1, 2, 0, 6, 6), (5, 1, 2, 6, 7), (7, 2, 3, 12, 11),
                                       (2, 1, 0, 5, 5)])
def test_dgrad_is_the_adjoint_of_linear(k, s, p, h, w):
    rng = np.random.default_rng(k * 100 + s * 10 + p)
    x = rng.standard_normal((3, 4, h, w))
    W = rng.standard_normal((5, 4, k, k))
    xt, Wt = t64(x, True), t64(W)
    y = TF.conv2d(xt, Wt, stride=s, padding=p)
    d = rng.standard_normal(tuple(y.shape))
    y.backward(t64(d))
    got = O.dgrad_plain(d, W, (h, w), s, p)
    assert np.max(np.abs(got - xt.grad.numpy())) < 1e-12
    # <dgrad(d), x> == <d, linear(x)>
    assert abs(np.sum(got * x) - np.sum(d * O.linear(W, x, s, p))) < 1e-9


def test_dgrad_fc():
    rng = np.random.default_rng(3)
    d, W = rng.standard_normal((4, 6)), rng.standard_normal((6, 9))
    assert np.allclose(O.dgrad_plain(d, W), d @ W)


def test_relu_and_pool_match_library_autograd_including_ties():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((2, 3, 6, 8))
    x[0, 0, :2, :2] = -1.0           # a window that ReLU turns into four equal zeros
    x[1, 2, 2:4, 4:6] = 0.75         # a window of four equal positive values
    xt = t64(x, True)
    y = TF.max_pool2d(TF.relu(xt), 2)
    assert np.array_equal(O.maxpool2x2(O.relu(x)), y.detach().numpy())
    dy = rng.standard_normal(tuple(y.shape))
    y.backward(t64(dy))
    got = O.relu_bwd(O.maxpool2x2_bwd(dy, O.relu(x)), x)
    assert np.max(np.abs(got - xt.grad.numpy())) < 1e-15
    # hand values: the gradient of a 2x2 window goes to its first maximum
    one = np.array([[[[1.0, 3.0], [3.0, 2.0]]]])
    assert np.array_equal(O.maxpool2x2_bwd(np.array([[[[5.0]]]]), one), np.array([[[[0.0, 5.0], [0.0, 0.0]]]]))


def test_training_step_matches_autograd_of_a_three_layer_chain():
    rng = np.random.default_rng(5)
    layers = [dict(stride=1, pad=1, pool=False, kh=3, kw=3), dict(stride=1, pad=1, pool=True, kh=3, kw=3),
              dict(stride=1, pad=1, pool=False, kh=3, kw=3)]
    chans = [3, 6, 6, 8]
    Ws = [rng.standard_normal((chans[i + 1], chans[i], 3, 3)) * (2.0 / (9 * chans[i])) ** 0.5 for i in range(3)]
    x0 = rng.random((4, 3, 8, 8))
    Wt = [t64(W, True) for W in Ws]
    a = t64(x0)
    for L, W in zip(layers, Wt):
        a = TF.relu(TF.conv2d(a, W, stride=L["stride"], padding=L["pad"]))
        if L["pool"]:
            a = TF.max_pool2d(a, 2)
    dL = rng.standard_normal(tuple(a.shape))
    a.backward(t64(dL))
    out = O.training_step_plain(layers, Ws, x0, dL, scale=0.25)
    assert np.max(np.abs(out["acts"][-1] - a.detach().numpy())) < 1e-12
    for W, dW in zip(Wt, out["dWs"]):
        assert np.max(np.abs(dW - 0.25 * W.grad.numpy())) < 1e-12


def test_weight_gradients_of_virtual_batches_add_up():
    """Section 6, 'Large Batch Aggregation': the batch gradient is the sum over virtual batches, so two
    calls on halves of the groups (the second adding to the first) give the whole."""
    spec = synth.LayerSpec("tiny", "t", "conv", 4, 5, 6, 6, 3, 3, 1, 1, K=2, G=4)
    d = synth.draw_layer(spec)
    xbar = O.encode(d["x"], d["r"], d["C"])
    whole = O.wgrad_masked(d["delta"], xbar, d["C"], d["gamma"], 0.125, 3, 3, 1, 1)
    K, E = spec.K, spec.K + 2
    parts = 0.0
    for lo, hi in ((0, 1), (1, 4)):
        parts = parts + O.wgrad_masked(d["delta"][lo * K:hi * K], xbar[lo * E:hi * E], d["C"][lo:hi],
                                       d["gamma"][lo:hi], 0.125, 3, 3, 1, 1)
    plain = O.wgrad_plain(d["delta"], d["x"], 0.125, 3, 3, 1, 1)
    assert np.max(np.abs(parts - whole)) < 1e-9 * np.max(np.abs(xbar))
    assert np.max(np.abs(parts - plain)) < 1e-9 * np.max(np.abs(xbar))
