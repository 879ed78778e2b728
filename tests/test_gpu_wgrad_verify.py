"""GPU parity of dk_linear_bwd_wgrad_verify against the oracle's redundant
weight-gradient check: the gradient itself within 1e-3 of the plain
definition, a clean verdict on honest results, and a single wrong element in
either of the two results flagged exactly at its index."""
import numpy as np
import pytest
import torch

from oracle import dk_oracle as O
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu

TOL_DECODED = 1e-3
TAU_W = 1e-2          # flagged iff not(|dW - dW_second| <= TAU_W * rms(dW))


def tiny(kind="conv", **kw):
    base = dict(workload="tiny", name="wv", kind=kind, cin=8, cout=12, K=2, G=2, sigma_r=100.0)
    if kind == "conv":
        base.update(h=9, w=7, kh=3, kw=3, stride=1, pad=1)
    base.update(kw)
    return synth.LayerSpec(**base)


CASES = [
    ("conv_tiny_K2", tiny()),
    ("fc_K4", tiny("fc", cin=64, cout=40, K=4, G=3)),
    ("conv_pair_K4", tiny(cin=64, cout=256, h=8, w=8, K=4, G=2)),
    ("conv_packed_taps_cin48", tiny(cin=48, cout=64, h=10, w=10, K=4, G=2)),
    ("conv_s2", tiny(cin=16, cout=24, h=11, w=11, stride=2, K=3, G=2)),
    ("stem_cin3", tiny(cin=3, cout=16, h=12, w=12, K=4, G=2)),
    ("vgg_cifar_conv3_1_G2", synth.layer("vgg16_cifar", "conv3_1").with_groups(2)),
]


@pytest.fixture(scope="module")
def ctx():
    c = dk.Context(0)
    yield c
    c.close()


def lay(spec):
    return dk.DK_NHWC


def flat_dw_index(spec, co, ci, u, v):
    """Index of a weight-gradient element as the device stores it ([cout][kh][kw][cin], or [cout][cin])."""
    if spec.kind == "fc":
        return co * spec.cin + ci
    return ((co * spec.kh + u) * spec.kw + v) * spec.cin + ci


@pytest.mark.parametrize("name,spec", CASES, ids=[c[0] for c in CASES])
def test_wgrad_verify_matches_oracle(ctx, name, spec):
    d = synth.draw_layer(spec)
    E = spec.K + 2
    p = dk.problem_from_spec(spec)
    ctx.ensure_workspace(p)
    xbar32 = O.encode(d["x"], d["r"], d["C"]).astype(np.float32)
    scale = 1.0 / spec.batch
    delta_d, xbar_d = H.acts_to_dev(d["delta"], lay(spec)), H.acts_to_dev(xbar32, lay(spec))
    dW = H.empty_weights(spec, lay(spec))
    v = dk.new_verdict()
    want = O.wgrad_redundant(d["delta"], xbar32, d["C"], d["gamma"], scale, spec.kh, spec.kw, spec.stride, spec.pad,
                             tau_w=TAU_W)
    assert not want["flags"].any()
    plain = O.wgrad_plain(d["delta"], d["x"], scale, spec.kh, spec.kw, spec.stride, spec.pad)

    dW.fill_(float("nan"))
    dk.dk_linear_bwd_wgrad_verify(ctx, p, delta_d, xbar_d, d["C"], d["gamma"], scale, TAU_W, dW, v)
    got_v = dk.read_verdict(v)
    assert (got_v["ok"], got_v["n_flagged"], got_v["first_index"], got_v["status"]) == (1, 0, -1, 0)
    assert got_v["max_ratio"] < TAU_W / 4          # honest difference of the two fp32-class results
    got = H.weights_from_dev(dW, lay(spec))
    assert H.max_rel(got, plain) < TOL_DECODED
    assert H.max_rel(got, want["dW"]) < TOL_DECODED
    # the plain entry point gives the same first result
    dW1 = torch.empty_like(dW)
    dk.dk_linear_bwd_wgrad(ctx, p, delta_d, xbar_d, E, d["C"], d["gamma"], scale, dW1)
    assert float((dW - dW1).abs().max()) <= 1e-4 * float(dW1.abs().max())

    # one wrong element in either result: flagged once, at its index
    co, ci = spec.cout - 1, spec.cin // 2
    u, w_ = (spec.kh - 1, 0) if spec.kind == "conv" else (0, 0)
    idx = (co, ci) if spec.kind == "fc" else (co, ci, u, w_)
    flat = flat_dw_index(spec, co, ci, u, w_)
    for which in (0, 1):
        val = 0.5 * want["rms"]
        bad = O.wgrad_redundant(d["delta"], xbar32, d["C"], d["gamma"], scale, spec.kh, spec.kw, spec.stride,
                                spec.pad, tau_w=TAU_W, fault=(which, idx, val))
        assert bad["flags"].sum() == 1 and bad["flags"][idx]
        # no element of the oracle's comparison sits near the threshold
        assert not ((bad["ratio"] > TAU_W / 4) & (bad["ratio"] < TAU_W * 4)).any()
        f = dk.dk_fault(0, which, flat, val)
        dk.dk_linear_bwd_wgrad_verify(ctx, p, delta_d, xbar_d, d["C"], d["gamma"], scale, TAU_W, dW, v, f)
        got_v = dk.read_verdict(v)
        assert (got_v["ok"], got_v["n_flagged"], got_v["first_index"]) == (0, 1, flat)
        assert got_v["max_ratio"] == pytest.approx(float(bad["ratio"].max()), rel=2e-2)
    assert dk.dk_device_status(ctx) == 0


def test_argument_checks(ctx):
    spec = tiny()
    p = dk.problem_from_spec(spec)
    ctx.ensure_workspace(p)
    d = synth.draw_layer(spec)
    dW = H.empty_weights(spec, lay(spec))
    v = dk.new_verdict()
    delta_d = H.acts_to_dev(d["delta"], lay(spec))
    xbar_d = H.acts_to_dev(O.encode(d["x"], d["r"], d["C"]).astype(np.float32), lay(spec))
    with pytest.raises(dk.DkError):          # tolerance must be positive
        dk.dk_linear_bwd_wgrad_verify(ctx, p, delta_d, xbar_d, d["C"], d["gamma"], 1.0, 0.0, dW, v)
    with pytest.raises(dk.DkError):          # fault outside dW
        dk.dk_linear_bwd_wgrad_verify(ctx, p, delta_d, xbar_d, d["C"], d["gamma"], 1.0, TAU_W, dW, v,
                                      dk.dk_fault(0, 0, dW.numel(), 1.0))
    odd = tiny("fc", cin=37, cout=19, K=1, G=3)          # n_in not a multiple of 4
    po = dk.problem_from_spec(odd)
    ctx.ensure_workspace(po)
    do = synth.draw_layer(odd)
    with pytest.raises(dk.DkError):
        dk.dk_linear_bwd_wgrad_verify(ctx, po, H.acts_to_dev(do["delta"], lay(odd)),
                                      H.acts_to_dev(O.encode(do["x"], do["r"], do["C"]).astype(np.float32), lay(odd)),
                                      do["C"], do["gamma"], 1.0, TAU_W, H.empty_weights(odd, lay(odd)), v)
