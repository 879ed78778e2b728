"""A tensor-core call served by several launches over ranges of virtual batches (the pre-pass of a later range
runs on the context's second stream beside the GEMM of an earlier one) gives the results of the single-launch
call: decoded outputs and stored encodings bit for bit (the tiles and their arithmetic are the same), the
weight gradient to within the error of its arithmetic (the contraction is sliced differently), verdicts identical; and both match the oracle."""
import numpy as np
import pytest
import torch

from oracle import dk_oracle as O
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu

TOL_DECODED = 1e-3


def spec_of(**kw):
    base = dict(workload="tiny", name="t", kind="conv", cin=16, cout=32, h=32, w=32, kh=3, kw=3, stride=1, pad=1,
                K=2, G=10, sigma_r=100.0)
    base.update(kw)
    return synth.LayerSpec(**base)


# enough tiles to fill the device without slicing the contraction (slices and ranges exclude each other)
CASES = [
    ("two_row_tiles_K2", spec_of()),
    ("single_cta_K3", spec_of(cin=32, cout=128, K=3, G=14, h=24, w=24)),
    ("pair_K2_cout256", spec_of(cin=32, cout=256, K=2, G=20, h=32, w=32)),
    ("pair_K4_groups_per_tile", spec_of(cin=32, cout=256, K=4, G=192, h=4, w=4)),
    ("fc_K4", synth.LayerSpec(workload="tiny", name="t", kind="fc", cin=256, cout=512, K=4, G=1280, sigma_r=100.0)),
]


@pytest.fixture()
def ctx():
    c = dk.Context(0)
    yield c
    c.close()


def launches(ctx, kind):
    return dk.dk_profile_read(ctx)[kind][2]


@pytest.mark.parametrize("nslab", [2, 3, 8])
@pytest.mark.parametrize("name,spec", CASES, ids=[c[0] for c in CASES])
def test_forward_in_ranges_equals_single_launch_and_oracle(ctx, name, spec, nslab):
    d = synth.draw_layer(spec)
    K, E, lay = spec.K, spec.K + 2, dk.DK_NHWC
    p = dk.problem_from_spec(spec, tol=H.TAU)
    ctx.ensure_workspace(p)
    W = H.weights_to_dev(d["W"], lay)
    x, r = H.acts_to_dev(d["x"], lay), H.acts_to_dev(d["r"], lay)
    v = dk.new_verdict()
    out = {}
    for n in (1, nslab):
        dk.dk_set_option(ctx, dk.DK_OPT_SLABS, 8)
        dk.dk_set_option(ctx, dk.DK_OPT_SLABS_FORCE, n)
        y = H.empty_acts(spec.G * K, spec, "out", lay)
        xsave = H.empty_acts(spec.G * E, spec, "in", lay)
        y.fill_(float("nan")); xsave.fill_(float("nan"))
        dk.dk_profile_reset(ctx)
        dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, xsave, v)
        torch.cuda.synchronize()
        out[n] = (y, xsave, dk.read_verdict(v), launches(ctx, "linear_fwd"))
    assert out[1][3] == 1 and 2 <= out[nslab][3] <= nslab
    assert torch.equal(out[1][0], out[nslab][0])
    assert torch.equal(out[1][1], out[nslab][1])
    got_v = out[nslab][2]
    assert (got_v["ok"], got_v["n_flagged"], got_v["first_index"], got_v["status"]) == (1, 0, -1, 0)
    assert got_v["max_ratio"] == pytest.approx(out[1][2]["max_ratio"], rel=1e-4)   # (sums of squares meet by atomics)
    plain = O.linear_plain(d["W"], d["x"], spec.stride, spec.pad)
    assert H.max_rel(H.acts_from_dev(out[nslab][0], lay), plain) < TOL_DECODED
    want_xbar = O.encode(d["x"], d["r"], d["C"])
    assert H.max_rel(H.acts_from_dev(out[nslab][1], lay), want_xbar) < 1e-6

    # a wrong accelerator output in the first, a middle and the last virtual batch: flagged once, at its place
    ybar = O.linear(d["W"], want_xbar.astype(np.float32), spec.stride, spec.pad)
    y2 = torch.empty_like(out[1][0])
    for g in (0, spec.G // 2, spec.G - 1):
        enc, co = (g % E), spec.cout - 1
        delta = 0.5 * float(np.sqrt(np.mean(ybar[g * E + enc] ** 2)))
        f = dk.dk_fault(g, enc, H.flat_out_index(spec, lay, co, spec.hout - 1, 0), delta)
        dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y2, None, v, f)
        got = dk.read_verdict(v)
        assert (got["ok"], got["n_flagged"], got["first_index"]) == (0, 1, g * spec.n_out + f.out_index)


@pytest.mark.parametrize("nslab", [2, 5])
@pytest.mark.parametrize("name,spec", CASES[:4], ids=[c[0] for c in CASES[:4]])
def test_wgrad_in_ranges_equals_single_launch_and_oracle(ctx, name, spec, nslab):
    d = synth.draw_layer(spec)
    K, E, lay = spec.K, spec.K + 2, dk.DK_NHWC
    p = dk.problem_from_spec(spec)
    ctx.ensure_workspace(p)
    xbar32 = O.encode(d["x"], d["r"], d["C"]).astype(np.float32)
    scale = 1.0 / spec.batch
    delta, xbar = H.acts_to_dev(d["delta"], lay), H.acts_to_dev(xbar32, lay)
    got = {}
    for n in (1, nslab):
        dk.dk_set_option(ctx, dk.DK_OPT_SLABS, 8)
        dk.dk_set_option(ctx, dk.DK_OPT_SLABS_FORCE, n)
        dW = H.empty_weights(spec, lay)
        dW.fill_(float("nan"))
        dk.dk_profile_reset(ctx)
        dk.dk_linear_bwd_wgrad(ctx, p, delta, xbar, E, d["C"], d["gamma"], scale, dW)
        torch.cuda.synchronize()
        assert dk.dk_device_status(ctx) == 0
        got[n] = (H.weights_from_dev(dW, lay), launches(ctx, "wgrad"))
    assert got[1][1] == 1 and 2 <= got[nslab][1] <= nslab
    # (other contraction slices, hence other chunk boundaries and another order of the atomics: the two agree to
    # within the arithmetic's own error, not bit for bit)
    assert H.max_rel(got[nslab][0], got[1][0]) < 5e-4
    plain = O.wgrad_plain(d["delta"], d["x"], scale, spec.kh, spec.kw, spec.stride, spec.pad)
    assert H.max_rel(got[nslab][0], plain) < TOL_DECODED

    # adding into an existing gradient: the first range must not clear it
    dW = H.weights_to_dev(np.full(got[1][0].shape, 2.0, dtype=np.float32), lay)
    dk.dk_linear_bwd_wgrad_accumulate(ctx, p, delta, xbar, E, d["C"], d["gamma"], scale, dW)
    assert H.max_rel(H.weights_from_dev(dW, lay) - 2.0, plain) < TOL_DECODED


def test_library_picks_the_number_of_ranges_when_allowed(ctx):
    """With DK_OPT_SLABS > 1 the library cuts a layer whose pre-pass is long against one round of GEMM tiles into
    ranges by itself, and a small one not; by default every call is one pre-pass and one GEMM launch."""
    for spec, several in ((synth.layer("vgg16_224", "conv2_1").with_groups(8), True),
                          (synth.layer("vgg16_cifar", "conv4_1").with_groups(2), False)):
        d = synth.draw_layer(spec, with_delta=False)
        lay = dk.DK_NHWC
        p = dk.problem_from_spec(spec, tol=H.TAU)
        ctx.ensure_workspace(p)
        y = H.empty_acts(spec.G * spec.K, spec, "out", lay)
        v = dk.new_verdict()
        W, x, r = H.weights_to_dev(d["W"], lay), H.acts_to_dev(d["x"], lay), H.acts_to_dev(d["r"], lay)
        for allowed in (1, 8):
            dk.dk_set_option(ctx, dk.DK_OPT_SLABS, allowed)
            dk.dk_profile_reset(ctx)
            dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, None, v)
            got = dk.read_verdict(v)
            assert (got["ok"], got["status"]) == (1, 0)
            n = launches(ctx, "linear_fwd")
            assert (n >= 2) if (several and allowed > 1) else (n == 1)


@pytest.mark.parametrize("name,cout", [("single_cta", 128), ("cta_pairs", 256)])
def test_paced_forward_gives_the_same_bits(ctx, name, cout):
    """DK_OPT_TC_PACE only decides when a CTA starts its next tiles: outputs, stored encodings and the verdict of a
    call whose CTAs walk many rounds of tiles are the same with the meetings off, at every tile and at the default."""
    spec = spec_of(cin=32, cout=cout, h=56, w=56, K=4, G=24)      # 2352 tiles (x 1 M tile): 16 or 32 rounds
    d = synth.draw_layer(spec, with_delta=False)
    lay = dk.DK_NHWC
    p = dk.problem_from_spec(spec, tol=H.TAU)
    ctx.ensure_workspace(p)
    W, x, r = H.weights_to_dev(d["W"], lay), H.acts_to_dev(d["x"], lay), H.acts_to_dev(d["r"], lay)
    v = dk.new_verdict()
    out = {}
    for every in (0, 1, 8):
        dk.dk_set_option(ctx, dk.DK_OPT_TC_PACE, every)
        y = H.empty_acts(spec.G * spec.K, spec, "out", lay)
        xsave = H.empty_acts(spec.G * (spec.K + 2), spec, "in", lay)
        y.fill_(float("nan")); xsave.fill_(float("nan"))
        dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, xsave, v)
        torch.cuda.synchronize()
        got = dk.read_verdict(v)
        assert (got["ok"], got["n_flagged"], got["status"]) == (1, 0, 0)
        assert dk.dk_device_status(ctx) == 0
        out[every] = (y, xsave)
    for every in (1, 8):
        assert torch.equal(out[0][0], out[every][0])
        assert torch.equal(out[0][1], out[every][1])
    plain = O.linear_plain(d["W"], d["x"][:4], spec.stride, spec.pad)
    assert H.max_rel(H.acts_from_dev(out[8][0], lay)[:4], plain) < TOL_DECODED
