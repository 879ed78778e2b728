"""GPU parity for the colluding-accelerator scheme (M noise vectors, S = K + M
encodings plus the redundant one).  The library has no separate entry point
for it: a virtual batch of K_lib = K + M - 1 "inputs" whose last M - 1 rows are
noise, plus the usual noise tensor, IS that scheme (the CPU pins show the
equivalence).  Here the C-ABI calls run on such inputs and are compared with
the oracle's Section 4.5 functions and with the plain definitions over the K
private inputs."""
import numpy as np
import pytest
import torch

from oracle import dk_oracle as O
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu

TOL_DECODED = 1e-3
TOL_ENCODE = 1e-6


def spec_for(kind, K, M, **kw):
    base = dict(workload="tiny", name="colluding", kind=kind, cin=32, cout=48, K=K + M - 1, G=3, sigma_r=100.0)
    if kind == "conv":
        base.update(h=10, w=9, kh=3, kw=3, stride=1, pad=1)
    base.update(kw)
    return synth.LayerSpec(**base)


CASES = [
    ("conv_K3_M2_pair", spec_for("conv", 3, 2, cin=64, cout=256, h=8, w=8), 3, 2),     # K_lib = 4, CTA pairs
    ("conv_K2_M2_single", spec_for("conv", 2, 2), 2, 2),                               # K_lib = 3, single CTA
    ("fc_K2_M3", spec_for("fc", 2, 3, cin=96, cout=40), 2, 3),                         # K_lib = 4
    ("conv_K1_M4_stem", spec_for("conv", 1, 4, cin=3, cout=16, h=12, w=12), 1, 4),     # K_lib = 4, 3-channel stem
]


@pytest.fixture(scope="module")
def ctx():
    c = dk.Context(0)
    yield c
    c.close()


def lay(spec):
    return dk.DK_NHWC


@pytest.mark.parametrize("name,spec,K,M", CASES, ids=[c[0] for c in CASES])
def test_forward_decodes_the_private_inputs(ctx, name, spec, K, M):
    d = synth.draw_colluding(spec, K, M)
    KL, S, E = spec.K, K + M, spec.K + 2
    p = dk.problem_from_spec(spec, tol=H.TAU)
    ctx.ensure_workspace(p)
    W = H.weights_to_dev(d["W"], lay(spec))
    x, r = H.acts_to_dev(d["x"], lay(spec)), H.acts_to_dev(d["r"], lay(spec))
    y = H.empty_acts(spec.G * KL, spec, "out", lay(spec))
    xsave = H.empty_acts(spec.G * E, spec, "in", lay(spec))
    v = dk.new_verdict()
    dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, xsave, v)
    got_v = dk.read_verdict(v)
    assert (got_v["ok"], got_v["n_flagged"], got_v["first_index"], got_v["status"]) == (1, 0, -1, 0)
    got_y = H.acts_from_dev(y, lay(spec))
    got_xbar = H.acts_from_dev(xsave, lay(spec))
    for g in range(spec.G):
        want_y = O.linear_plain(d["W"], d["x_private"][g], spec.stride, spec.pad)
        # relative to the scale of the outputs of the whole call
        assert H.max_rel(got_y[g * KL:g * KL + K], want_y) < TOL_DECODED
        want_xbar = O.encode_colluding(d["x_private"][g], d["R"][g], d["A1"][g], d["A2"][g])
        assert H.max_rel(got_xbar[g * E:g * E + S], want_xbar) < TOL_ENCODE
        # the rows that stand for noise decode to <W, r_m>, which the caller drops
        want_z = O.linear(d["W"], d["R"][g][:M - 1], spec.stride, spec.pad)
        if M > 1:
            assert H.max_rel(got_y[g * KL + K:(g + 1) * KL], want_z) < TOL_DECODED

    # one wrong encoded output is flagged at its coordinate
    clean = O.masked_forward(d["W"], d["x"], d["r"], d["C"], spec.stride, spec.pad, H.TAU)
    g, enc = spec.G - 1, S - 1
    co, oh, ow = spec.cout - 1, spec.hout - 1, 0
    row = g * E + enc
    delta = 0.5 * float(np.sqrt(np.mean(clean["ybar"][row] ** 2)))
    bad = O.masked_forward(d["W"], d["x"], d["r"], d["C"], spec.stride, spec.pad, H.TAU,
                           fault=(row, H.logical_out_index(spec, co, oh, ow), delta))
    H.assert_no_gray_zone(bad["ratio"])
    f = dk.dk_fault(g, enc, H.flat_out_index(spec, lay(spec), co, oh, ow), delta)
    dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, None, v, f)
    got_v = dk.read_verdict(v)
    assert (got_v["ok"], got_v["n_flagged"], got_v["first_index"]) == (0, 1, g * spec.n_out + f.out_index)


@pytest.mark.parametrize("name,spec,K,M", CASES, ids=[c[0] for c in CASES])
def test_weight_gradient_of_the_private_inputs(ctx, name, spec, K, M):
    d = synth.draw_colluding(spec, K, M)
    E = spec.K + 2
    p = dk.problem_from_spec(spec)
    ctx.ensure_workspace(p)
    xbar32 = O.encode(d["x"], d["r"], d["C"]).astype(np.float32)
    scale = 1.0 / (spec.G * K)
    dW = H.empty_weights(spec, lay(spec))
    dW.fill_(float("nan"))
    dk.dk_linear_bwd_wgrad(ctx, p, H.acts_to_dev(d["delta"], lay(spec)), H.acts_to_dev(xbar32, lay(spec)),
                           E, d["C"], d["gamma"], scale, dW)
    assert dk.dk_device_status(ctx) == 0
    got = H.weights_from_dev(dW, lay(spec))
    xp = d["x_private"].reshape((spec.G * K,) + d["x_private"].shape[2:])
    dp = d["delta_private"].reshape((spec.G * K,) + d["delta_private"].shape[2:])
    plain = O.wgrad_plain(dp, xp, scale, spec.kh, spec.kw, spec.stride, spec.pad)
    assert H.max_rel(got, plain) < TOL_DECODED
    total = None
    for g in range(spec.G):
        xbar = O.encode_colluding(d["x_private"][g], d["R"][g], d["A1"][g], d["A2"][g])
        part = O.wgrad_colluding(d["delta_private"][g], xbar, d["A1"][g], d["A2"][g], d["gamma"][g], scale,
                                 spec.kh, spec.kw, spec.stride, spec.pad)
        total = part if total is None else total + part
    assert H.max_rel(got, total) < TOL_DECODED


# also through the kernels that are not the tensor-core epilogue: fp32 SIMT (channels-first would do too), the
# fp64 regime's fused pointwise kernel and its general path
SKIP_CASES = CASES + [
    ("pw_K2_M2_fp64_fused", spec_for("conv", 2, 2, cin=32, cout=48, h=6, w=6, kh=1, kw=1, pad=0, precision="fp64"), 2, 2),
    ("conv_K2_M2_fp64", spec_for("conv", 2, 2, cin=8, cout=12, h=6, w=6, precision="fp64"), 2, 2),
]


@pytest.mark.parametrize("name,spec,K,M", SKIP_CASES, ids=[c[0] for c in SKIP_CASES])
def test_outputs_of_the_noise_rows_are_not_stored_when_told_so(ctx, name, spec, K, M):
    """DK_OPT_NOISE_ROWS = M - 1: the rows of y that would hold <W, r_m> stay as they were, the private rows
    and the verdict are those of the default call (fused call, and dk_decode_verify on the same y_bar)."""
    d = synth.draw_colluding(spec, K, M)
    KL, E = spec.K, spec.K + 2
    p = dk.problem_from_spec(spec, tol=H.TAU)
    ctx.ensure_workspace(p)
    W = H.weights_to_dev(d["W"], lay(spec))
    x, r = H.acts_to_dev(d["x"], lay(spec)), H.acts_to_dev(d["r"], lay(spec))
    v = dk.new_verdict()
    y_all = H.empty_acts(spec.G * KL, spec, "out", lay(spec))
    dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y_all, None, v)
    want_v = dk.read_verdict(v)
    xbar = H.acts_to_dev(O.encode(d["x"], d["r"], d["C"]).astype(np.float32), lay(spec))
    ybar = H.empty_acts(spec.G * E, spec, "out", lay(spec))
    dk.dk_linear_fwd(ctx, p, W, xbar, ybar)
    try:
        dk.dk_set_option(ctx, dk.DK_OPT_NOISE_ROWS, M - 1)
        sentinel = -12345.0
        for call in ("fused", "decode"):
            y = H.empty_acts(spec.G * KL, spec, "out", lay(spec))
            y.fill_(sentinel)
            if call == "fused":
                dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, None, v)
            else:
                dk.dk_decode_verify(ctx, p, ybar, d["C"], None, y, v)
            got_v = dk.read_verdict(v)
            assert (got_v["ok"], got_v["n_flagged"], got_v["status"]) == (want_v["ok"], want_v["n_flagged"], 0)
            yv, ya = y.reshape(spec.G, KL, -1), y_all.reshape(spec.G, KL, -1)
            assert bool((yv[:, K:] == sentinel).all()), call
            # (small problems meet by atomic additions in y_bar: equal up to that order)
            assert float((yv[:, :K] - ya[:, :K]).abs().max()) <= 1e-4 * float(ya.abs().max()), call
    finally:
        dk.dk_set_option(ctx, dk.DK_OPT_NOISE_ROWS, 0)
