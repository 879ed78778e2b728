"""Parity at full size, in the launch configuration the benchmark times: EVERY
layer of all five workloads (`fc784`, `vgg16_cifar`, `resnet18_224`,
`mobilenetv2_pw`, `vgg16_224` at batch 256) through dk_masked_linear (encodings
stored) and, where the workload trains, dk_linear_bwd_wgrad.

The oracle cannot run a whole layer of the large workloads in a test, so the
decoded outputs are compared on a seeded sample of at least 4096 output
coordinates (image corners, first and last group and channel, and the very
last element of the tensor always among them) and the weight gradient on at
least 256 coordinates, each evaluated one by one from the plain definition.
Properties that hold at any size complete the check: a clean verdict on the
honest run, exactly one flagged element at the right index under one injected
fault, and stored encodings equal to Eq. 1 of the inputs.

Inputs are drawn on the host by the seeded generators; moving them to the
device, permuting them to channels-last and gathering the sampled outputs are
plain copies."""
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

SPECS = [s for wl in ("fc784", "vgg16_cifar", "resnet18_224", "mobilenetv2_pw", "vgg16_224") for s in synth.layers(wl)]


@pytest.fixture(scope="module")
def ctx():
    c = dk.Context(0)
    yield c
    c.close()


def to_dev(a):
    """Logical host array -> device tensor in the library's channels-last layout (the permutation runs on
    the device; a 4-D weight array [cout, cin, kh, kw] becomes [cout, kh, kw, cin])."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    if t.ndim == 4:
        t = t.permute(0, 2, 3, 1).contiguous()
    return t


def sampled_y_error(spec, d, y_dev):
    coords = synth.sample_coordinates(spec, 2 * N_Y, "y")      # duplicates are dropped by the sampler
    K = spec.K
    ks = np.random.default_rng(5).integers(0, K, len(coords))
    # the last element of the whole tensor: last sample, channel and pixel
    coords = np.concatenate([coords, [[spec.G - 1, spec.cout - 1, spec.hout - 1, spec.wout - 1]]])
    ks = np.concatenate([ks, [K - 1]])
    b = coords[:, 0] * K + ks
    bi, ci, hi, wi = (torch.from_numpy(v.astype(np.int64)).cuda() for v in (b, coords[:, 1], coords[:, 2], coords[:, 3]))
    got = (y_dev[bi, ci] if spec.kind == "fc" else y_dev[bi, hi, wi, ci]).cpu().numpy().astype(np.float64)
    W64 = d["W"].astype(np.float64)
    want = np.array([O.linear_at(W64, d["x"][bb], co, oh, ow, spec.stride, spec.pad)
                     for bb, (_, co, oh, ow) in zip(b, coords)])
    assert len(want) >= min(N_Y, spec.G * spec.n_out)
    return float(np.max(np.abs(got - want)) / np.max(np.abs(want)))


def sampled_dw_error(spec, d, dW_dev, scale_arg):
    coords = synth.sample_coordinates(spec, 2 * N_DW, "dw")
    coords = coords[np.lexsort((coords[:, 1], coords[:, 0]))]
    got_all = dW_dev.cpu().numpy()         # [cout, kh, kw, cin] or [cout, cin]
    assert len(coords) >= min(N_DW, spec.cout * spec.kc)
    worst, scale = 0.0, 0.0
    for (co, ci, u, v) in coords:
        want = O.wgrad_plain_at(d["delta"], d["x"], scale_arg, co, ci, u, v, spec.stride, spec.pad)
        got = got_all[co, ci] if spec.kind == "fc" else got_all[co, u, v, ci]
        worst = max(worst, abs(float(got) - want))
        scale = max(scale, abs(want))
    return worst / scale


@pytest.mark.parametrize("spec", SPECS, ids=[f"{s.workload}:{s.name}" for s in SPECS])
def test_full_size_layer_matches_oracle_on_samples(ctx, spec):
    d = synth.draw_layer(spec, with_delta=spec.wgrad)
    K, E = spec.K, spec.K + 2
    p = dk.problem_from_spec(spec, tol=H.TAU)
    ctx.ensure_workspace(p)
    W, x, r = to_dev(d["W"]), to_dev(d["x"]), to_dev(d["r"])
    y = H.empty_acts(spec.batch, spec, "out", dk.DK_NHWC)
    xsave = H.empty_acts(spec.G * E, spec, "in", dk.DK_NHWC)
    v = dk.new_verdict()
    dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, xsave, v)
    vd = dk.read_verdict(v)
    assert (vd["ok"], vd["n_flagged"], vd["first_index"], vd["status"]) == (1, 0, -1, 0)
    assert vd["max_ratio"] < H.TAU / 4
    assert sampled_y_error(spec, d, y) < TOL_DECODED

    # the stored encodings are Eq. 1 of the inputs (first and last row)
    for row in (0, spec.G * E - 1):
        g, i = divmod(row, E)
        want = O.encode(d["x"][g * K:(g + 1) * K], d["r"][g:g + 1], d["C"][g:g + 1])[i]
        got = H.acts_from_dev(xsave[row:row + 1], dk.DK_NHWC)
        assert H.max_rel(H.read_positions(spec, got), H.read_positions(spec, want[None])) < 1e-6

    # one wrong accelerator output, last group, last encoding, last position of the tensor
    g, enc = spec.G - 1, E - 1
    co, oh, ow = spec.cout - 1, spec.hout - 1, spec.wout - 1
    xb_row = O.encode(d["x"][g * K:(g + 1) * K], d["r"][g:g + 1], d["C"][g:g + 1])[enc]
    ybar_row_rms = float(np.sqrt(np.mean(O.linear(d["W"], xb_row[None], spec.stride, spec.pad) ** 2)))
    f = dk.dk_fault(g, enc, H.flat_out_index(spec, dk.DK_NHWC, co, oh, ow), 0.5 * ybar_row_rms)
    dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, None, v, f)
    vd = dk.read_verdict(v)
    assert (vd["ok"], vd["n_flagged"], vd["first_index"]) == (0, 1, g * spec.n_out + f.out_index)
    assert f.out_index == spec.n_out - 1

    if spec.wgrad:
        dW = H.empty_weights(spec, dk.DK_NHWC)
        scale = 1.0 / spec.batch
        delta = to_dev(d["delta"])
        dk.dk_linear_bwd_wgrad(ctx, p, delta, xsave, E, d["C"], d["gamma"], scale, dW)
        assert dk.dk_device_status(ctx) == 0
        assert sampled_dw_error(spec, d, dW, scale) < TOL_DECODED
    del W, x, r, y, xsave
    torch.cuda.empty_cache()


X2_SPECS = [synth.layer("vgg16_cifar", "conv1_2"), synth.layer("vgg16_cifar", "conv4_2"), synth.layer("resnet18_224", "layer2_3x3s2"),
            synth.layer("resnet18_224", "layer4_3x3"), synth.layer("vgg16_224", "conv3_2"), synth.layer("vgg16_224", "conv5_1"),
            synth.layer("vgg16_224", "fc6"), synth.layer("vgg16_224", "fc8")]


@pytest.mark.parametrize("spec", X2_SPECS, ids=[f"{s.workload}:{s.name}" for s in X2_SPECS])
def test_full_size_forward_with_unsplit_weights(ctx, spec):
    """DK_TF32X2_WUNSPLIT (W as one TF32 term, two products per step) at full size: sampled decoded outputs
    within 5e-4 of the oracle (the bar the mode is offered under), clean verdict, fault flagged."""
    d = synth.draw_layer(spec, with_delta=False)
    E = spec.K + 2
    p = dk.problem_from_spec(spec, precision=dk.DK_TF32X2_WUNSPLIT, tol=H.TAU)
    ctx.ensure_workspace(p)
    W, x, r = to_dev(d["W"]), to_dev(d["x"]), to_dev(d["r"])
    y = H.empty_acts(spec.batch, spec, "out", dk.DK_NHWC)
    v = dk.new_verdict()
    dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, None, v)
    vd = dk.read_verdict(v)
    assert (vd["ok"], vd["n_flagged"], vd["first_index"], vd["status"]) == (1, 0, -1, 0)
    assert vd["max_ratio"] < H.TAU / 4
    assert sampled_y_error(spec, d, y) < 5e-4
    f = dk.dk_fault(1, 2, spec.n_out // 3, 500.0)
    dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, None, v, f)
    vd = dk.read_verdict(v)
    assert (vd["ok"], vd["n_flagged"], vd["first_index"]) == (0, 1, 1 * spec.n_out + f.out_index)
    del W, x, r, y
    torch.cuda.empty_cache()
