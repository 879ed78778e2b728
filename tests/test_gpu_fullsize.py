"""Parity at the benchmark's full sizes and launch configuration: every layer
of the `vgg16_cifar` workload (batch 128, K = 4, 32 virtual batches) through
dk_masked_linear (encodings stored) and dk_linear_bwd_wgrad, compared with the
oracle on seeded samples of output coordinates (each evaluated one by one from
the plain definition), plus the properties that hold at any size: a clean
verdict, and exactly one flagged element at the right index under one injected
fault.  One layer of each other workload family is checked the same way."""
import numpy as np
import pytest
import torch

from oracle import dk_oracle as O
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu

TOL_DECODED = 1e-3
N_Y, N_DW = 4096, 256

VGG = synth.layers("vgg16_cifar")
OTHERS = [synth.layer("resnet18_224", "layer3_3x3"), synth.layer("resnet18_224", "layer2_ds"),
          synth.layer("mobilenetv2_pw", "expand_96_576"), synth.layer("mobilenetv2_pw", "project_960_320"),
          synth.layer("vgg16_224", "fc7"), synth.layer("vgg16_224", "conv5_1")]


@pytest.fixture(scope="module")
def ctx():
    c = dk.Context(0)
    yield c
    c.close()


def _sampled_y_error(spec, d, y_dev):
    coords = synth.sample_coordinates(spec, N_Y, "y")
    got_all = y_dev.cpu().numpy()          # [batch, ho, wo, cout] or [batch, cout]
    K = spec.K
    worst, scale = 0.0, 0.0
    rng = np.random.default_rng(5)
    ks = rng.integers(0, K, len(coords))
    for (g, co, oh, ow), k in zip(coords, ks):
        b = g * K + k
        want = O.linear_at(d["W"], d["x"][b], co, oh, ow, spec.stride, spec.pad)
        got = got_all[b, co] if spec.kind == "fc" else got_all[b, oh, ow, co]
        worst = max(worst, abs(float(got) - want))
        scale = max(scale, abs(want))
    return worst / scale


def _sampled_dw_error(spec, d, dW_dev, scale_arg):
    coords = synth.sample_coordinates(spec, N_DW, "dw")
    got_all = dW_dev.cpu().numpy()         # [cout, kh, kw, cin] or [cout, cin]
    worst, scale = 0.0, 0.0
    for (co, ci, u, v) in coords:
        want = O.wgrad_plain_at(d["delta"], d["x"], scale_arg, co, ci, u, v, spec.stride, spec.pad)
        got = got_all[co, ci] if spec.kind == "fc" else got_all[co, u, v, ci]
        worst = max(worst, abs(float(got) - want))
        scale = max(scale, abs(want))
    return worst / scale


@pytest.mark.parametrize("spec", VGG + OTHERS, ids=[f"{s.workload}:{s.name}" for s in VGG + OTHERS])
def test_full_size_layer_matches_oracle_on_samples(ctx, spec):
    d = synth.draw_layer(spec, with_delta=spec.wgrad)
    K, E = spec.K, spec.K + 2
    p = dk.problem_from_spec(spec, tol=H.TAU)
    ctx.ensure_workspace(p)
    W = H.weights_to_dev(d["W"], dk.DK_NHWC)
    x, r = H.acts_to_dev(d["x"], dk.DK_NHWC), H.acts_to_dev(d["r"], dk.DK_NHWC)
    y = H.empty_acts(spec.batch, spec, "out", dk.DK_NHWC)
    xsave = H.empty_acts(spec.G * E, spec, "in", dk.DK_NHWC)
    v = dk.new_verdict()
    dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, xsave, v)
    vd = dk.read_verdict(v)
    assert (vd["ok"], vd["n_flagged"], vd["first_index"], vd["status"]) == (1, 0, -1, 0)
    assert vd["max_ratio"] < H.TAU / 4
    assert _sampled_y_error(spec, d, y) < TOL_DECODED

    # the stored encodings are Eq. 1 of the inputs (spot check of two rows)
    for row in (0, spec.G * E - 1):
        g, i = divmod(row, E)
        want = O.encode(d["x"][g * K:(g + 1) * K], d["r"][g:g + 1], d["C"][g:g + 1])[i]
        got = H.acts_from_dev(xsave[row:row + 1], dk.DK_NHWC)[0]
        assert H.max_rel(got, want) < 1e-6

    # one wrong accelerator output, last group, last position
    g, enc = spec.G - 1, E - 1
    co, oh, ow = spec.cout - 1, spec.hout - 1, spec.wout - 1
    xb_row = O.encode(d["x"][g * K:(g + 1) * K], d["r"][g:g + 1], d["C"][g:g + 1])[enc]
    ybar_row_rms = float(np.sqrt(np.mean(O.linear(d["W"], xb_row[None], spec.stride, spec.pad) ** 2)))
    f = dk.dk_fault(g, enc, H.flat_out_index(spec, dk.DK_NHWC, co, oh, ow), 0.5 * ybar_row_rms)
    dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, None, v, f)
    vd = dk.read_verdict(v)
    assert (vd["ok"], vd["n_flagged"], vd["first_index"]) == (0, 1, g * spec.n_out + f.out_index)

    if spec.wgrad:
        dW = H.empty_weights(spec, dk.DK_NHWC)
        scale = 1.0 / spec.batch
        dk.dk_linear_bwd_wgrad(ctx, p, H.acts_to_dev(d["delta"], dk.DK_NHWC), xsave, E, d["C"], d["gamma"],
                               scale, dW)
        assert dk.dk_device_status(ctx) == 0
        assert _sampled_dw_error(spec, d, dW, scale) < TOL_DECODED
    torch.cuda.empty_cache()
