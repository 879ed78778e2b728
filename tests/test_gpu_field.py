"""GPU parity of the finite-field calls (Section 5, Algorithm 1) against the
exact CPU oracle on the same seeded inputs.  Everything here is integer work:
residues, decoded integers, verdicts and the dequantised outputs (exact
multiples of 2^-l) must match bit for bit."""
import numpy as np
import pytest
import torch

from oracle import dk_field_oracle as F
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu

P = F.P_PAPER
L = F.L_PAPER


def tiny(kind="conv", **kw):
    base = dict(workload="tiny_field", name="t", kind=kind, cin=8, cout=12, K=2, G=2)
    if kind == "conv":
        base.update(h=9, w=7, kh=3, kw=3, stride=1, pad=1)
    base.update(kw)
    return synth.LayerSpec(**base)


CASES = [
    ("fc784", synth.layers("fc784")[0], dk.DK_NHWC),
    ("fc_ragged_K1", tiny("fc", cin=37, cout=19, K=1, G=3), dk.DK_NHWC),
    ("fc_K8_long", tiny("fc", cin=20011, cout=70, K=8, G=1), dk.DK_NHWC),     # several reductions per sum
    ("fc_long_tc", tiny("fc", cin=20012, cout=130, K=2, G=1), dk.DK_NHWC),    # tcgen05 kernel, sliced contraction
    # 1025 k-tiles in 16 slices of 65: each slice folds its class sums once before its end
    ("fc_very_long_tc", tiny("fc", cin=131076, cout=8, K=1, G=1), dk.DK_NHWC),
    ("conv_tiny_K2", tiny(), dk.DK_NHWC),
    ("conv_ragged_K3_nchw", tiny(cin=5, cout=7, h=6, w=5, K=3, G=2), dk.DK_NCHW),
    ("conv_7x7s2_stem", tiny(cin=3, cout=16, h=20, w=20, kh=7, kw=7, stride=2, pad=3, K=4, G=1), dk.DK_NHWC),
    ("conv_1x1s2", tiny(cin=16, cout=24, h=10, w=10, kh=1, kw=1, stride=2, pad=0, K=4, G=2), dk.DK_NHWC),
    ("conv_3x3s2_K5", tiny(cin=12, cout=20, h=11, w=11, stride=2, K=5, G=1), dk.DK_NHWC),
    ("vgg_cifar_conv3_1_G2", synth.layer("vgg16_cifar", "conv3_1").with_groups(2), dk.DK_NHWC),
    ("vgg_cifar_conv5_1_G2", synth.layer("vgg16_cifar", "conv5_1").with_groups(2), dk.DK_NHWC),
    ("mbv2_project_960_320_G1", synth.layer("mobilenetv2_pw", "project_960_320").with_groups(1), dk.DK_NHWC),
    # operands fetched by TMA from digit planes (channels-last, stride 1, cin % 64 == 0): 64- and 128-byte rows,
    # ragged pixel boxes, ragged output channels, no padding, a 5x5 filter
    ("conv_tma_cin64", tiny(cin=64, cout=72, h=9, w=7, K=2, G=2), dk.DK_NHWC),
    ("conv_tma_cin128_5x5", tiny(cin=128, cout=130, h=6, w=10, kh=5, kw=5, pad=2, K=3, G=1), dk.DK_NHWC),
    ("conv_tma_cin192_nopad", tiny(cin=192, cout=16, h=8, w=8, pad=0, K=1, G=3), dk.DK_NHWC),
    ("fc_tma_cin640", tiny("fc", cin=640, cout=200, K=4, G=5), dk.DK_NHWC),
]


def res_dev(a: np.ndarray) -> torch.Tensor:
    """Residues (int64 on the host, all below 2^31) -> int32 device tensor."""
    return torch.from_numpy(np.ascontiguousarray(a).astype(np.int32)).cuda()


def res_acts_to_dev(a, layout):
    if a.ndim == 4 and layout == dk.DK_NHWC:
        a = a.transpose(0, 2, 3, 1)
    return res_dev(a)


def res_acts_from_dev(t, layout):
    a = t.cpu().numpy().astype(np.int64)
    if a.ndim == 4 and layout == dk.DK_NHWC:
        a = a.transpose(0, 3, 1, 2)
    return a


def res_weights_to_dev(W, layout):
    if W.ndim == 4 and layout == dk.DK_NHWC:
        W = W.transpose(0, 2, 3, 1)
    return res_dev(W)


def res_weights_from_dev(t, layout):
    W = t.cpu().numpy().astype(np.int64)
    if W.ndim == 4 and layout == dk.DK_NHWC:
        W = W.transpose(0, 3, 1, 2)
    return W


def empty_res(like: torch.Tensor) -> torch.Tensor:
    return torch.empty(like.shape, dtype=torch.int32, device="cuda")


def u32(a):
    return np.ascontiguousarray(a, dtype=np.uint32)


@pytest.fixture(scope="module")
def ctx():
    c = dk.Context(0)
    yield c
    c.close()


def test_quantize_matches_round_and_field(ctx):
    rng = np.random.default_rng(5)
    v = np.concatenate([rng.uniform(-300, 300, 100003), rng.standard_normal(5000) * 1e-3,
                        np.array([0.0, 0.5, -0.5, 1.5, -1.5, 2.5, 0.001953125, -0.001953125, 0.005859375,
                                  131071.998, -131072.0, 1e7, -1e7, 3.0e11, -3.0e11])]).astype(np.float32)
    t = torch.from_numpy(v).cuda()
    out = torch.empty(v.shape, dtype=torch.int32, device="cuda")
    for bits in (L, 2 * L, 0):
        dk.dk_field_quantize(ctx, t, bits, P, out)
        assert np.array_equal(out.cpu().numpy().astype(np.int64), F.quantize(v, bits, P)), bits
    # the way back: centred residue times 2^-bits
    back = torch.empty(v.shape, dtype=torch.float32, device="cuda")
    dk.dk_field_quantize(ctx, t, L, P, out)
    dk.dk_field_dequantize(ctx, out, L, P, back)
    want = F.centre(F.quantize(v, L, P), P).astype(np.float64) / 2 ** L
    assert np.array_equal(back.cpu().numpy().astype(np.float64), want)


@pytest.mark.parametrize("name,spec,layout", CASES, ids=[c[0] for c in CASES])
def test_unfused_calls_match_the_oracle(ctx, name, spec, layout):
    d = synth.draw_field_layer(spec, P)
    p = dk.problem_from_spec(spec, layout=layout)
    E = spec.K + 2
    Wq, xq, bq = F.quantize(d["W"], L, P), F.quantize(d["x"], L, P), F.quantize(d["bias"], 2 * L, P)
    C = u32(d["Cq"])

    # quantise on the device, from the same fp32 tensors
    x_dev = H.acts_to_dev(d["x"], layout)
    xq_dev = empty_res(x_dev)
    dk.dk_field_quantize(ctx, x_dev, L, P, xq_dev)
    assert np.array_equal(res_acts_from_dev(xq_dev, layout), xq)

    # Eq. 1
    rq_dev = res_acts_to_dev(d["rq"], layout)
    xbar_dev = torch.empty((spec.G * E,) + tuple(xq_dev.shape[1:]), dtype=torch.int32, device="cuda")
    dk.dk_field_encode(ctx, p, P, xq_dev, rq_dev, C, xbar_dev)
    want_xbar = F.field_encode(xq, d["rq"], d["Cq"], P)
    assert np.array_equal(res_acts_from_dev(xbar_dev, layout), want_xbar)

    # the linear operation on the encodings
    Wq_dev = res_weights_to_dev(Wq, layout)
    ybar_dev = torch.empty(H.empty_acts(spec.G * E, spec, "out", layout).shape, dtype=torch.int32, device="cuda")
    dk.dk_field_linear_fwd(ctx, p, P, Wq_dev, xbar_dev, ybar_dev)
    want_ybar = F.field_linear(Wq, want_xbar, P, spec.stride, spec.pad)
    assert np.array_equal(res_acts_from_dev(ybar_dev, layout), want_ybar)

    # Eq. 2, the redundant equation, bias, centring, Round
    yq_dev = torch.empty(H.empty_acts(spec.batch, spec, "out", layout).shape, dtype=torch.int32, device="cuda")
    y_dev = H.empty_acts(spec.batch, spec, "out", layout)
    v = dk.new_verdict()
    dk.dk_field_decode_verify(ctx, p, P, L, ybar_dev, C, res_dev(bq), yq_dev, y_dev, v)
    yq, zq = F.field_decode(want_ybar, d["Cq"], P)
    assert np.array_equal(yq, F.field_linear_plain(Wq, xq, P, spec.stride, spec.pad))
    shape = (1, -1) + (1,) * (yq.ndim - 2)
    want_yc = F.centre((yq + bq.reshape(shape)) % P, P)
    assert np.array_equal(res_acts_from_dev(yq_dev, layout), want_yc)
    assert np.array_equal(H.acts_from_dev(y_dev, layout).astype(np.float64), F.dequantize_output(want_yc, L))
    got = dk.read_verdict(v)
    assert (got["ok"], got["n_flagged"], got["first_index"], got["status"]) == (1, 0, -1, 0)

    # a tampered accelerator output: one residue of y_bar changed on the device
    g, enc = spec.G - 1, (spec.K + 1) if spec.K % 2 else 0
    e = (spec.n_out * 2) // 3
    flat = ybar_dev.view(spec.G * E, -1)
    flat[g * E + enc, e] = (int(flat[g * E + enc, e]) + 12345) % P
    dk.dk_field_decode_verify(ctx, p, P, L, ybar_dev, C, None, yq_dev, None, v)
    tampered = H.mem_order(want_ybar, layout).reshape(spec.G * E, -1).copy()
    tampered[g * E + enc, e] = (tampered[g * E + enc, e] + 12345) % P
    tampered = tampered.reshape(H.mem_order(want_ybar, layout).shape)
    y2, z2 = F.field_decode(tampered, d["Cq"], P)
    want_v = F.field_verdict(F.field_verify(tampered, d["Cq"], y2, z2, P))
    got = dk.read_verdict(v)
    assert {k: got[k] for k in want_v} == want_v == {"ok": 0, "n_flagged": 1, "first_index": g * spec.n_out + e}


@pytest.mark.parametrize("name,spec,layout", CASES, ids=[c[0] for c in CASES])
def test_masked_linear_and_wgrad_match_the_oracle(ctx, name, spec, layout):
    d = synth.draw_field_layer(spec, P)
    p = dk.problem_from_spec(spec, layout=layout)
    ctx.ensure_workspace(p, field=True)
    E = spec.K + 2
    C, gamma = u32(d["Cq"]), u32(d["gammaq"])
    W_dev, x_dev = H.weights_to_dev(d["W"], layout), H.acts_to_dev(d["x"], layout)
    rq_dev = res_acts_to_dev(d["rq"], layout)
    bias_dev = H.dev(d["bias"])
    y_dev = H.empty_acts(spec.batch, spec, "out", layout)
    yq_dev = torch.empty(y_dev.shape, dtype=torch.int32, device="cuda")
    xsave = torch.empty((spec.G * E,) + tuple(x_dev.shape[1:]), dtype=torch.int32, device="cuda")
    v = dk.new_verdict()
    dk.dk_field_masked_linear(ctx, p, P, L, W_dev, x_dev, rq_dev, C, bias_dev, y_dev, yq_dev, xsave, v)
    want = F.field_masked_forward(d["W"], d["x"], d["rq"], d["Cq"], L, P, spec.stride, spec.pad, bias=d["bias"])
    assert np.array_equal(res_acts_from_dev(xsave, layout), want["xbar"])
    assert np.array_equal(res_acts_from_dev(yq_dev, layout), want["yq"])
    assert np.array_equal(H.acts_from_dev(y_dev, layout).astype(np.float64), want["y"])
    got = dk.read_verdict(v)
    assert (got["ok"], got["n_flagged"], got["first_index"]) == (1, 0, -1) and not want["flags"].any()

    # one wrong accelerator output through the library's own hook
    g, enc, e = 0, spec.K, spec.n_out - 1
    f = dk.dk_field_fault(g, enc, e, P - 1)
    dk.dk_field_masked_linear(ctx, p, P, L, W_dev, x_dev, rq_dev, C, None, None, yq_dev, None, v, f)
    got = dk.read_verdict(v)
    assert (got["ok"], got["n_flagged"], got["first_index"]) == (0, 1, g * spec.n_out + e)

    # Eq. 4-6: quantised output gradients, stored encodings, decoded exactly
    delta_dev = H.acts_to_dev(d["delta"], layout)
    dq_dev = empty_res(delta_dev)
    dk.dk_field_quantize(ctx, delta_dev, L, P, dq_dev)
    dWq_dev = torch.empty(H.empty_weights(spec, layout).shape, dtype=torch.int32, device="cuda")
    dk.dk_field_linear_bwd_wgrad(ctx, p, P, dq_dev, xsave, E, C, gamma, dWq_dev)
    dq = F.quantize(d["delta"], L, P)
    want_dw = F.field_wgrad_masked(dq, want["xbar"], d["Cq"], d["gammaq"], P, spec.kh, spec.kw, spec.stride,
                                   spec.pad)
    assert np.array_equal(res_weights_from_dev(dWq_dev, layout), want_dw)
    assert np.array_equal(want_dw, F.field_wgrad_plain(dq, want["xq"], P, spec.kh, spec.kw, spec.stride, spec.pad))
    # back to floating point: centred residue * 2^-2l
    dW_dev = H.empty_weights(spec, layout)
    dk.dk_field_dequantize(ctx, dWq_dev, 2 * L, P, dW_dev)
    assert np.array_equal(H.weights_from_dev(dW_dev, layout).astype(np.float64),
                          F.centre(want_dw, P).astype(np.float64) / 4 ** L)


@pytest.mark.parametrize("prime", [65537, 2 ** 27 - 39, 2 ** 29 - 3])
@pytest.mark.parametrize("kind", ["fc", "conv"])
def test_other_primes(ctx, prime, kind):
    """Any odd prime below 2^30 is served: a small one (the decoded integers wrap, parity is modulo p all the
    same), the largest one below 2^27 (the last to take the short reduction in the elementwise kernels) and one
    above it (64-bit reductions everywhere)."""
    spec = tiny("fc", cin=300, cout=21, K=3, G=2) if kind == "fc" else tiny(cin=6, cout=10, h=7, w=6, K=8, G=1)
    d = synth.draw_field_layer(spec, prime)
    p = dk.problem_from_spec(spec)
    ctx.ensure_workspace(p, field=True)
    E = spec.K + 2
    C, gamma = u32(d["Cq"]), u32(d["gammaq"])
    W_dev, x_dev = H.weights_to_dev(d["W"], dk.DK_NHWC), H.acts_to_dev(d["x"], dk.DK_NHWC)
    rq_dev = res_acts_to_dev(d["rq"], dk.DK_NHWC)
    y_dev = H.empty_acts(spec.batch, spec, "out", dk.DK_NHWC)
    yq_dev = torch.empty(y_dev.shape, dtype=torch.int32, device="cuda")
    xsave = torch.empty((spec.G * E,) + tuple(x_dev.shape[1:]), dtype=torch.int32, device="cuda")
    v = dk.new_verdict()
    dk.dk_field_masked_linear(ctx, p, prime, L, W_dev, x_dev, rq_dev, C, H.dev(d["bias"]), y_dev, yq_dev, xsave, v)
    want = F.field_masked_forward(d["W"], d["x"], d["rq"], d["Cq"], L, prime, spec.stride, spec.pad, bias=d["bias"])
    assert np.array_equal(res_acts_from_dev(xsave, dk.DK_NHWC), want["xbar"])
    assert np.array_equal(res_acts_from_dev(yq_dev, dk.DK_NHWC), want["yq"])
    assert np.array_equal(H.acts_from_dev(y_dev, dk.DK_NHWC).astype(np.float64), want["y"])
    assert dk.read_verdict(v)["ok"] == 1
    f = dk.dk_field_fault(spec.G - 1, spec.K + 1, 5, 1)
    dk.dk_field_masked_linear(ctx, p, prime, L, W_dev, x_dev, rq_dev, C, None, None, yq_dev, None, v, f)
    got = dk.read_verdict(v)
    assert (got["ok"], got["n_flagged"], got["first_index"]) == (0, 1, (spec.G - 1) * spec.n_out + 5)
    delta_dev = H.acts_to_dev(d["delta"], dk.DK_NHWC)
    dq_dev = empty_res(delta_dev)
    dk.dk_field_quantize(ctx, delta_dev, L, prime, dq_dev)
    dWq_dev = torch.empty(H.empty_weights(spec, dk.DK_NHWC).shape, dtype=torch.int32, device="cuda")
    dk.dk_field_linear_bwd_wgrad(ctx, p, prime, dq_dev, xsave, E, C, gamma, dWq_dev)
    dq = F.quantize(d["delta"], L, prime)
    assert np.array_equal(res_weights_from_dev(dWq_dev, dk.DK_NHWC),
                          F.field_wgrad_plain(dq, want["xq"], prime, spec.kh, spec.kw, spec.stride, spec.pad))


def test_argument_errors_are_reported_without_launching(ctx):
    spec = tiny("fc", cin=8, cout=4, K=2, G=1)
    p = dk.problem_from_spec(spec)
    t = torch.zeros(16, dtype=torch.float32, device="cuda")
    o = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(dk.DkError) as ei:
        dk.dk_field_quantize(ctx, t, L, 2 ** 25 - 37, o)        # not a prime
    assert ei.value.status == 1
    d = synth.draw_field_layer(spec, P)
    C = u32(d["Cq"]).copy()
    C[0, 1] = C[0, 0]                                            # singular square part
    v = dk.new_verdict()
    ybar = torch.zeros((4, 4), dtype=torch.int32, device="cuda")
    yq = torch.zeros((2, 4), dtype=torch.int32, device="cuda")
    with pytest.raises(dk.DkError) as ei:
        dk.dk_field_decode_verify(ctx, p, P, L, ybar, C, None, yq, None, v)
    assert ei.value.status == 3


@pytest.mark.parametrize("layer", ["conv2_2", "conv5_1"])
def test_full_size_layer_sampled_against_the_oracle(ctx, layer):
    """A whole layer of the CIFAR-shaped VGG-16 workload (all 32 virtual batches, the
    configuration `bench.py --field-table` times): decoded integers and weight-gradient
    residues at sampled coordinates against single elements computed in Python integers;
    the verdict must be clean and an injected fault found."""
    spec = synth.layer("vgg16_cifar", layer)
    d = synth.draw_field_layer(spec, P)
    p = dk.problem_from_spec(spec)
    ctx.ensure_workspace(p, field=True)
    E = spec.K + 2
    C, gamma = u32(d["Cq"]), u32(d["gammaq"])
    W_dev, x_dev = H.weights_to_dev(d["W"], dk.DK_NHWC), H.acts_to_dev(d["x"], dk.DK_NHWC)
    rq_dev = res_acts_to_dev(d["rq"], dk.DK_NHWC)
    yq_dev = torch.empty(H.empty_acts(spec.batch, spec, "out", dk.DK_NHWC).shape, dtype=torch.int32, device="cuda")
    xsave = torch.empty((spec.G * E,) + tuple(x_dev.shape[1:]), dtype=torch.int32, device="cuda")
    v = dk.new_verdict()
    dk.dk_field_masked_linear(ctx, p, P, L, W_dev, x_dev, rq_dev, C, None, None, yq_dev, xsave, v)
    got = dk.read_verdict(v)
    assert (got["ok"], got["n_flagged"], got["first_index"]) == (1, 0, -1)
    Wq, xq = F.quantize(d["W"], L, P), F.quantize(d["x"], L, P)
    yq = res_acts_from_dev(yq_dev, dk.DK_NHWC)
    for g, co, oh, ow in synth.sample_coordinates(spec, 24, "y"):
        for k in (0, spec.K - 1):
            s = int(g) * spec.K + k
            want = F.centre(np.array(F.field_linear_at(Wq, xq[s], co, oh, ow, P, spec.stride, spec.pad)), P)
            assert yq[s, co, oh, ow] == want
    f = dk.dk_field_fault(spec.G - 1, 1, 77, 1)
    dk.dk_field_masked_linear(ctx, p, P, L, W_dev, x_dev, rq_dev, C, None, None, yq_dev, None, v, f)
    got = dk.read_verdict(v)
    assert (got["ok"], got["n_flagged"], got["first_index"]) == (0, 1, (spec.G - 1) * spec.n_out + 77)

    delta_dev = H.acts_to_dev(d["delta"], dk.DK_NHWC)
    dq_dev = empty_res(delta_dev)
    dk.dk_field_quantize(ctx, delta_dev, L, P, dq_dev)
    dWq_dev = torch.empty(H.empty_weights(spec, dk.DK_NHWC).shape, dtype=torch.int32, device="cuda")
    dk.dk_field_linear_bwd_wgrad(ctx, p, P, dq_dev, xsave, E, C, gamma, dWq_dev)
    dWq = res_weights_from_dev(dWq_dev, dk.DK_NHWC)
    dq = F.quantize(d["delta"], L, P)
    for co, ci, u, vv in synth.sample_coordinates(spec, 12, "dw"):
        assert dWq[co, ci, u, vv] == F.field_wgrad_plain_at(dq, xq, co, ci, u, vv, P, spec.stride, spec.pad)


CROSS_CHECK = [c for c in CASES if c[0] in ("conv_tiny_K2", "fc_K8_long", "conv_3x3s2_K5", "conv_ragged_K3_nchw",
                                            "vgg_cifar_conv3_1_G2", "fc_long_tc", "conv_tma_cin64")]


@pytest.mark.parametrize("path", [1, 2, 3], ids=["integer_alu", "mma_sync", "tcgen05_register_split"])
@pytest.mark.parametrize("name,spec,layout", CROSS_CHECK, ids=[c[0] for c in CROSS_CHECK])
def test_cross_check_kernels_give_the_same_residues(name, spec, layout, path):
    """Option DK_OPT_FIELD_PATH = 1 selects the 64-bit integer-ALU contraction kernels, 2 keeps the
    contractions on the mma.sync kernels instead of the tcgen05 ones, 3 keeps them off the TMA-fed tcgen05
    kernels: the encoded outputs and the weight gradient are the same residues as the oracle's under each."""
    c = dk.Context(0)
    try:
        dk.dk_set_option(c, dk.DK_OPT_FIELD_PATH, path)
        d = synth.draw_field_layer(spec, P)
        p = dk.problem_from_spec(spec, layout=layout)
        c.ensure_workspace(p, field=True)
        E = spec.K + 2
        Wq, xq = F.quantize(d["W"], L, P), F.quantize(d["x"], L, P)
        xbar = F.field_encode(xq, d["rq"], d["Cq"], P)
        want_ybar = F.field_linear(Wq, xbar, P, spec.stride, spec.pad)
        ybar_dev = empty_res(res_acts_to_dev(want_ybar, layout))
        dk.dk_field_linear_fwd(c, p, P, res_weights_to_dev(Wq, layout), res_acts_to_dev(xbar, layout), ybar_dev)
        assert np.array_equal(res_acts_from_dev(ybar_dev, layout), want_ybar)
        dq = F.quantize(d["delta"], L, P)
        dWq = empty_res(res_weights_to_dev(Wq, layout))
        dk.dk_field_linear_bwd_wgrad(c, p, P, res_acts_to_dev(dq, layout), res_acts_to_dev(xbar, layout), E,
                                     u32(d["Cq"]), u32(d["gammaq"]), dWq)
        assert dk.dk_device_status(c) == 0
        assert np.array_equal(res_weights_from_dev(dWq, layout),
                              F.field_wgrad_plain(dq, xq, P, spec.kh, spec.kw, spec.stride, spec.pad))
    finally:
        c.close()


# ---------------------------------------------------------------------------
# Adversarial residues: every operand equal to p - 1, the value with the largest
# base-256 digits, at contraction lengths around the fold interval of the
# tensor-core kernels (8192 terms per class sum) and for a prime close to the
# 2^30 limit.  The expected results are closed forms in Python integers:
# (p-1)^2 = 1 (mod p), so a contraction of n such products is n mod p.
# ---------------------------------------------------------------------------
ADV_PRIMES = [2 ** 25 - 39, 2 ** 30 - 35]
# multiples of 4 take a tcgen05 kernel, multiples of 64 the TMA-fed one (64-byte rows; 128-byte rows for multiples of 128)
ADV_LENGTHS = [8188, 8191, 8192, 8193, 8196, 16380, 16385, 16388, 24580, 8128, 8256, 16320, 16384, 16448, 24640]


@pytest.mark.parametrize("prime", ADV_PRIMES)
@pytest.mark.parametrize("n", ADV_LENGTHS)
def test_linear_fwd_on_maximal_residues(ctx, prime, n):
    assert F.is_prime(prime)
    for cout, use_ws in ((130, True), (24, False)):           # tcgen05 kernel (workspace) / mma.sync kernel
        spec = tiny("fc", cin=n, cout=cout, K=2, G=1)
        p = dk.problem_from_spec(spec)
        if use_ws:
            ctx.ensure_workspace(p, field=True)
        Wq = torch.full((cout, n), prime - 1, dtype=torch.int64).to(torch.int32).cuda()
        xbar = torch.full((spec.G * (spec.K + 2), n), prime - 1, dtype=torch.int64).to(torch.int32).cuda()
        ybar = torch.empty((spec.G * (spec.K + 2), cout), dtype=torch.int32, device="cuda")
        dk.dk_field_linear_fwd(ctx, p, prime, Wq, xbar, ybar)
        assert dk.dk_device_status(ctx) == 0
        want = (n * pow(prime - 1, 2, prime)) % prime
        got = ybar.cpu().numpy().astype(np.int64) & 0xFFFFFFFF
        assert np.all(got == want), (prime, n, cout, int(got.flat[0]), want)


@pytest.mark.parametrize("prime", ADV_PRIMES)
@pytest.mark.parametrize("pixels", [8191, 8193, 16385])
def test_wgrad_on_maximal_residues(ctx, prime, pixels):
    """K = 1 with the identity as square coefficient block: B = [[1/gamma_0], [0]], so the mixed gradient of
    encoding 0 is delta itself and that of encoding 1 is zero.  With delta = x_bar = p - 1 everywhere the
    1x1 convolution's weight gradient is (number of pixels) * (p-1)^2 = pixels (mod p) in every element."""
    spec = tiny("conv", cin=16, cout=24, h=1, w=pixels, kh=1, kw=1, pad=0, K=1, G=1)
    p = dk.problem_from_spec(spec)
    ctx.ensure_workspace(p, field=True)
    C = np.array([[[1, 0], [0, 1], [5, 7]]], dtype=np.uint32)
    gamma = np.array([[3, 11]], dtype=np.uint32)
    dq = torch.full((1, 1, pixels, spec.cout), prime - 1, dtype=torch.int64).to(torch.int32).cuda()
    xbar = torch.full((3, 1, pixels, spec.cin), prime - 1, dtype=torch.int64).to(torch.int32).cuda()
    dWq = torch.empty((spec.cout, 1, 1, spec.cin), dtype=torch.int32, device="cuda")
    dk.dk_field_linear_bwd_wgrad(ctx, p, prime, dq, xbar, 3, C, gamma, dWq)
    assert dk.dk_device_status(ctx) == 0
    want = (pixels * pow(prime - 1, 2, prime)) % prime
    got = dWq.cpu().numpy().astype(np.int64) & 0xFFFFFFFF
    assert np.all(got == want), (prime, pixels, int(got.flat[0]), want)
    # the same through the oracle's own single-element routine
    d64 = np.full((1, spec.cout, 1, pixels), prime - 1, dtype=np.int64)
    x64 = np.full((1, spec.cin, 1, pixels), prime - 1, dtype=np.int64)
    assert F.field_wgrad_plain_at(d64, x64, 3, 5, 0, 0, prime, 1, 0) == want


@pytest.mark.parametrize("name,spec,layout", [c for c in CASES if c[1].K >= 2][:4],
                         ids=[c[0] for c in CASES if c[1].K >= 2][:4])
def test_noise_rows_are_not_decoded_when_told_so(ctx, name, spec, layout):
    """DK_OPT_NOISE_ROWS = n in the finite field (Section 4.5's relabelling): the last n decoded rows of every
    virtual batch keep what the buffers held, the other rows and the verdict are those of the default call."""
    d = synth.draw_field_layer(spec, P)
    p = dk.problem_from_spec(spec, layout=layout)
    ctx.ensure_workspace(p, field=True)
    K, n = spec.K, spec.K - 1
    C = u32(d["Cq"])
    W_dev, x_dev = H.weights_to_dev(d["W"], layout), H.acts_to_dev(d["x"], layout)
    rq_dev = res_acts_to_dev(d["rq"], layout)
    v = dk.new_verdict()
    y_all = H.empty_acts(spec.batch, spec, "out", layout)
    yq_all = torch.empty(y_all.shape, dtype=torch.int32, device="cuda")
    dk.dk_field_masked_linear(ctx, p, P, L, W_dev, x_dev, rq_dev, C, None, y_all, yq_all, None, v)
    want_v = dk.read_verdict(v)
    try:
        dk.dk_set_option(ctx, dk.DK_OPT_NOISE_ROWS, n)
        y = torch.full_like(y_all, -12345.0)
        yq = torch.full_like(yq_all, -12345)
        dk.dk_field_masked_linear(ctx, p, P, L, W_dev, x_dev, rq_dev, C, None, y, yq, None, v)
        got_v = dk.read_verdict(v)
        assert (got_v["ok"], got_v["n_flagged"], got_v["first_index"]) == \
               (want_v["ok"], want_v["n_flagged"], want_v["first_index"])
        for got, ref, sentinel in ((y, y_all, -12345.0), (yq, yq_all, -12345)):
            a, b = got.reshape(spec.G, K, -1), ref.reshape(spec.G, K, -1)
            assert bool((a[:, K - n:] == sentinel).all())
            assert torch.equal(a[:, :K - n], b[:, :K - n])
    finally:
        dk.dk_set_option(ctx, dk.DK_OPT_NOISE_ROWS, 0)
