"""GPU parity of the steps that chain the masked products into a training step
(Section 4.2 back-propagation of delta without encoding, the ReLU / MaxPool
layers of the Section 3.1 flow, Section 6 aggregation over virtual batches)
against the fp64 oracle on the same seeded inputs, and of a whole three-layer
VGG-style chain at CIFAR size: decoded activations, propagated gradients and
weight gradients within 1e-3 (max-norm relative), integrity verdicts clean."""
import numpy as np
import pytest
import torch

from oracle import dk_oracle as O
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu

TOL = 1e-3


@pytest.fixture(scope="module")
def ctx():
    c = dk.Context(0)
    yield c
    c.close()


def spec_of(kind="conv", **kw):
    base = dict(workload="tiny", name="t", kind=kind, cin=8, cout=12, K=2, G=2, sigma_r=100.0)
    if kind == "conv":
        base.update(h=9, w=7, kh=3, kw=3, stride=1, pad=1)
    base.update(kw)
    return synth.LayerSpec(**base)


DGRAD_CASES = [
    ("tc_3x3", spec_of(cin=16, cout=32, h=12, w=10, K=2, G=4)),
    ("tc_pair_cin256", spec_of(cin=256, cout=64, h=8, w=8, K=4, G=2)),
    ("tc_1x1", spec_of(cin=32, cout=24, h=6, w=6, kh=1, kw=1, pad=0, K=4, G=1)),
    ("tc_5x5_pad1", spec_of(cin=8, cout=8, h=9, w=9, kh=5, kw=5, pad=1, K=2, G=2)),
    ("tc_fc", spec_of("fc", cin=128, cout=72, K=4, G=3)),
    ("tc_batch_of_9", spec_of(cin=8, cout=16, h=6, w=6, K=3, G=3)),
    ("vgg_cifar_conv3_2_G2", synth.layer("vgg16_cifar", "conv3_2").with_groups(2)),
    ("simt_stride2", spec_of(cin=12, cout=20, h=11, w=11, stride=2, K=4, G=1)),
    ("simt_7x7s2", spec_of(cin=3, cout=16, h=20, w=20, kh=7, kw=7, stride=2, pad=3, K=4, G=1)),
    ("simt_1x1s2", spec_of(cin=16, cout=24, h=10, w=10, kh=1, kw=1, stride=2, pad=0, K=4, G=2)),
    ("simt_ragged_channels", spec_of(cin=5, cout=7, h=6, w=5, K=3, G=2)),
    ("simt_fc_ragged", spec_of("fc", cin=37, cout=19, K=1, G=3)),
]


@pytest.mark.parametrize("name,spec", DGRAD_CASES, ids=[c[0] for c in DGRAD_CASES])
def test_dgrad_matches_oracle(ctx, name, spec):
    d = synth.draw_layer(spec)
    p = dk.problem_from_spec(spec)
    ctx.ensure_workspace(p)
    W = H.weights_to_dev(d["W"], dk.DK_NHWC)
    delta = H.acts_to_dev(d["delta"], dk.DK_NHWC)
    dx = torch.full(H.empty_acts(spec.batch, spec, "in", dk.DK_NHWC).shape, float("nan"), device="cuda")
    dk.dk_profile_reset(ctx)
    dk.dk_linear_bwd_dgrad(ctx, p, W, delta, dx)
    assert dk.dk_device_status(ctx) == 0
    # the tensor-core form launches two preparation kernels (flipped filters, split of delta), the gather
    # kernel none: the case runs on the path its name says
    assert dk.dk_profile_read(ctx)["other"][2] == (0 if name.startswith("simt") else 2)
    want = O.dgrad_plain(d["delta"], d["W"], (spec.h, spec.w), spec.stride, spec.pad)
    assert H.max_rel(H.acts_from_dev(dx, dk.DK_NHWC), want) < 2e-5


def test_dgrad_nchw_layout(ctx):
    spec = spec_of(cin=6, cout=10, h=7, w=8, K=2, G=2)
    d = synth.draw_layer(spec)
    p = dk.problem_from_spec(spec, layout=dk.DK_NCHW)
    ctx.ensure_workspace(p)
    dx = torch.empty((spec.batch, spec.cin, spec.h, spec.w), device="cuda")
    dk.dk_linear_bwd_dgrad(ctx, p, H.dev(d["W"]), H.dev(d["delta"]), dx)
    want = O.dgrad_plain(d["delta"], d["W"], (spec.h, spec.w), spec.stride, spec.pad)
    assert H.max_rel(dx.cpu().numpy(), want) < 2e-5


@pytest.mark.parametrize("n,h,w,c", [(3, 8, 6, 16), (2, 7, 9, 12), (2, 6, 6, 5), (4, 1, 1, 40), (1, 32, 32, 64)])
@pytest.mark.parametrize("pool", [False, True])
def test_relu_pool_forward_and_backward_match_oracle(ctx, n, h, w, c, pool):
    if pool and (h < 2 or w < 2):
        pytest.skip("no 2x2 window")
    rng = np.random.default_rng(n * 1000 + h * 10 + c)
    x = rng.standard_normal((n, c, h, w)).astype(np.float32)
    x[0, 0, :2, :2] = -1.0                # a window ReLU turns into equal zeros
    if h >= 4 and w >= 4:
        x[0, 1, 2:4, 2:4] = 0.75          # a window of equal positive values: the first one takes the gradient
    he, we = (h // 2 * 2, w // 2 * 2) if pool else (h, w)
    want_y = O.maxpool2x2(O.relu(x[:, :, :he, :we])) if pool else O.relu(x)
    xd = H.acts_to_dev(x, dk.DK_NHWC)
    y = torch.empty((n, want_y.shape[2], want_y.shape[3], c), device="cuda")
    dk.dk_relu_pool_fwd(ctx, xd, n, h, w, c, pool, y)
    assert np.array_equal(H.acts_from_dev(y, dk.DK_NHWC), want_y.astype(np.float32))
    dy = rng.standard_normal(want_y.shape).astype(np.float32)
    dx = torch.full((n, h, w, c), float("nan"), device="cuda")
    dk.dk_relu_pool_bwd(ctx, H.acts_to_dev(dy, dk.DK_NHWC), xd, n, h, w, c, pool, dx)
    want_dx = np.zeros(x.shape)
    if pool:
        want_dx[:, :, :he, :we] = O.relu_bwd(O.maxpool2x2_bwd(dy, O.relu(x[:, :, :he, :we])), x[:, :, :he, :we])
    else:
        want_dx = O.relu_bwd(dy, x)
    assert np.array_equal(H.acts_from_dev(dx, dk.DK_NHWC), want_dx.astype(np.float32))


@pytest.mark.parametrize("spec", [spec_of(cin=16, cout=32, h=8, w=8, K=2, G=6),
                                  spec_of(cin=3, cout=16, h=10, w=10, K=4, G=3),
                                  spec_of("fc", cin=64, cout=40, K=4, G=5)], ids=["tc", "stem_simt", "fc"])
def test_weight_gradient_accumulates_over_slices_of_the_virtual_batches(ctx, spec):
    """Section 6, 'Large Batch Aggregation': a first call on some groups, then accumulating calls on the
    others, give the gradient of the whole batch."""
    d = synth.draw_layer(spec)
    K, E = spec.K, spec.K + 2
    xbar = O.encode(d["x"], d["r"], d["C"]).astype(np.float32)
    xb, dl = H.acts_to_dev(xbar, dk.DK_NHWC), H.acts_to_dev(d["delta"], dk.DK_NHWC)
    scale = 1.0 / spec.batch
    dW = torch.full(H.empty_weights(spec, dk.DK_NHWC).shape, float("nan"), device="cuda")
    cuts = [0, 1, spec.G // 2 + 1, spec.G]
    for i, (lo, hi) in enumerate(zip(cuts[:-1], cuts[1:])):
        p = dk.problem_from_spec(spec, G=hi - lo)
        ctx.ensure_workspace(dk.problem_from_spec(spec))
        args = (ctx, p, dl[lo * K:hi * K], xb[lo * E:hi * E], E, d["C"][lo:hi].copy(), d["gamma"][lo:hi].copy(),
                scale, dW)
        (dk.dk_linear_bwd_wgrad if i == 0 else dk.dk_linear_bwd_wgrad_accumulate)(*args)
    assert dk.dk_device_status(ctx) == 0
    want = O.wgrad_plain(d["delta"], d["x"], scale, spec.kh, spec.kw, spec.stride, spec.pad)
    assert H.max_rel(H.weights_from_dev(dW, dk.DK_NHWC), want) < TOL


# ---------------------------------------------------------------------------
# a three-layer VGG-style chain at CIFAR size, the GPU feeding itself
# ---------------------------------------------------------------------------
CHAIN = [dict(cin=3, cout=64, pool=False), dict(cin=64, cout=64, pool=True), dict(cin=64, cout=128, pool=False)]
CHAIN_K, CHAIN_G = 4, 2
KINK_BANDS = [1e-9, 1e-6, 1e-6]


def chain_specs():
    out, hw = [], 32
    for i, L in enumerate(CHAIN):
        out.append(synth.LayerSpec("chain3", f"conv{i}", "conv", L["cin"], L["cout"], hw, hw, 3, 3, 1, 1,
                                   K=CHAIN_K, G=CHAIN_G, sigma_r=100.0))
        if L["pool"]:
            hw //= 2
    return out


def chain_inputs(seed):
    specs = chain_specs()
    rng = np.random.default_rng(seed)
    per_layer = []
    for s in specs:
        per_layer.append({
            "W": (rng.standard_normal((s.cout, s.cin, 3, 3)) * np.sqrt(2.0 / s.kc)).astype(np.float32),
            "r": (rng.standard_normal((s.G, s.cin, s.h, s.w)) * s.sigma_r).astype(np.float32),
            "C": synth.draw_coefficients(rng, s.K, s.G), "gamma": synth.draw_gamma(rng, s.K, s.G)})
    x0 = rng.random((specs[0].batch, 3, 32, 32), dtype=np.float32)
    last = specs[-1]
    dL = rng.standard_normal((last.batch, last.cout, last.hout, last.wout)).astype(np.float32)
    return specs, per_layer, x0, dL


def oracle_chain(specs, per_layer, x0, dL):
    layers = [dict(stride=1, pad=1, pool=L["pool"], kh=3, kw=3) for L in CHAIN]
    return O.training_step_plain(layers, [p["W"] for p in per_layer], x0, dL, 1.0 / specs[0].batch)


def kink_free(ref, bands):
    """True when no ReLU input and no pooling decision of the oracle's step lies within the layer's band
    (relative to the layer's largest pre-activation) of its switching point: only then do the masks of a
    run with errors below the band provably equal the oracle's, and gradients can be compared element by
    element."""
    for L, z, band in zip(CHAIN, ref["pre"], bands):
        eps = band * float(np.max(np.abs(z)))
        if np.any(np.abs(z) < eps):
            return False
        if L["pool"]:
            a = O.relu(z)
            n, c, h, w = a.shape
            win = np.sort(a.reshape(n, c, h // 2, 2, w // 2, 2).transpose(0, 1, 2, 4, 3, 5).reshape(n, c, h // 2, w // 2, 4),
                          axis=4)
            gap = win[..., 3] - win[..., 2]
            if np.any((gap < eps) & (win[..., 3] > 0)):
                return False
    return True


def gpu_chain(ctx, specs, per_layer, x0, dL, precision, backward):
    dev_acts = [H.acts_to_dev(x0, dk.DK_NHWC)]
    pre, xsaves, verdicts, probs = [], [], [], []
    for s, P, L in zip(specs, per_layer, CHAIN):
        p = dk.problem_from_spec(s, precision=precision, tol=H.TAU)
        ctx.ensure_workspace(p)
        probs.append(p)
        z = H.empty_acts(s.batch, s, "out", dk.DK_NHWC)
        xs = H.empty_acts(s.G * (s.K + 2), s, "in", dk.DK_NHWC)
        v = dk.new_verdict()
        dk.dk_masked_linear(ctx, p, H.weights_to_dev(P["W"], dk.DK_NHWC), dev_acts[-1], H.acts_to_dev(P["r"], dk.DK_NHWC),
                            P["C"], None, z, xs, v)
        verdicts.append(dk.read_verdict(v))
        ho, wo = (s.hout // 2, s.wout // 2) if L["pool"] else (s.hout, s.wout)
        a = torch.empty((s.batch, ho, wo, s.cout), device="cuda")
        dk.dk_relu_pool_fwd(ctx, z, s.batch, s.hout, s.wout, s.cout, L["pool"], a)
        pre.append(z); xsaves.append(xs); dev_acts.append(a)
    out = {"acts": dev_acts, "pre": pre, "verdicts": verdicts, "deltas": [None] * len(specs), "dWs": [None] * len(specs)}
    if not backward:
        return out
    g = H.acts_to_dev(dL, dk.DK_NHWC)
    for li in range(len(specs) - 1, -1, -1):
        s, P, L = specs[li], per_layer[li], CHAIN[li]
        p = dk.problem_from_spec(s, tol=H.TAU)          # the backward products always run in the default arithmetic
        ctx.ensure_workspace(p)
        d = torch.empty_like(pre[li])
        dk.dk_relu_pool_bwd(ctx, g, pre[li], s.batch, s.hout, s.wout, s.cout, L["pool"], d)
        dW = H.empty_weights(s, dk.DK_NHWC)
        dk.dk_linear_bwd_wgrad(ctx, p, d, xsaves[li], s.K + 2, P["C"], P["gamma"], 1.0 / s.batch, dW)
        out["deltas"][li], out["dWs"][li] = d, dW
        if li > 0:
            g = H.empty_acts(s.batch, s, "in", dk.DK_NHWC)
            dk.dk_linear_bwd_dgrad(ctx, p, H.weights_to_dev(P["W"], dk.DK_NHWC), d, g)
    assert dk.dk_device_status(ctx) == 0
    return out


def test_chain_forward_in_the_default_arithmetic(ctx):
    """Decoded activations of every layer of the chain (each layer's input is the GPU's own previous
    output) within 1e-3 of the oracle's, every integrity verdict clean."""
    specs, per_layer, x0, dL = chain_inputs(20)
    ref = oracle_chain(specs, per_layer, x0, dL)
    got = gpu_chain(ctx, specs, per_layer, x0, dL, None, backward=False)
    for li in range(len(specs)):
        vd = got["verdicts"][li]
        assert (vd["ok"], vd["n_flagged"], vd["status"]) == (1, 0, 0)
        assert H.max_rel(H.acts_from_dev(got["pre"][li], dk.DK_NHWC), ref["pre"][li]) < TOL
        assert H.max_rel(H.acts_from_dev(got["acts"][li + 1], dk.DK_NHWC), ref["acts"][li + 1]) < TOL


def test_chain_training_step_matches_oracle(ctx):
    """The whole step, the GPU feeding itself: forward, ReLU/pool, gradient back-propagation and masked
    weight gradients.  ReLU and max pooling are discontinuous in their gradient, so an element-wise
    comparison of gradients needs identical switching decisions on both sides: the forward pass runs in
    the library's fp64 arithmetic and the inputs are redrawn (seeded) until the oracle has no
    pre-activation and no pooling decision within a band of its switching point.  The bands: the first
    layer sees identical fp32 inputs on both sides and the fp64 path is then off by ~1e-12 of the largest
    pre-activation (band 1e-9); the later layers see the GPU's own activations, stored in fp32 (each off
    by up to 6e-8 of itself, ~1e-8 of the largest pre-activation after the contraction: band 1e-6).
    The backward products (weight gradient on the stored encodings, delta propagation) run in the default
    tensor-core arithmetic and are continuous in their inputs."""
    for seed in range(30, 400):
        specs, per_layer, x0, dL = chain_inputs(seed)
        ref = oracle_chain(specs, per_layer, x0, dL)
        if kink_free(ref, KINK_BANDS):
            break
    else:
        pytest.fail("no kink-free draw found")
    got = gpu_chain(ctx, specs, per_layer, x0, dL, dk.DK_FP64_SIMT, backward=True)
    for li in range(len(specs)):
        vd = got["verdicts"][li]
        assert (vd["ok"], vd["n_flagged"], vd["status"]) == (1, 0, 0)
        assert H.max_rel(H.acts_from_dev(got["pre"][li], dk.DK_NHWC), ref["pre"][li]) < 1e-6
        assert H.max_rel(H.acts_from_dev(got["deltas"][li], dk.DK_NHWC), ref["deltas"][li]) < TOL
        assert H.max_rel(H.weights_from_dev(got["dWs"][li], dk.DK_NHWC), ref["dWs"][li]) < TOL
