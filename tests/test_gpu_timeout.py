"""Failure handling of the pipelined tensor-core kernels, exercised without
faulting or hanging the GPU: every wait inside them is bounded, and a kernel
whose wait runs out stops, reports DK_ERR_TIMEOUT and leaves the context
usable.  The test makes a wait run out in the permitted way: a host-set option
makes the producer of the next launch arm one pipeline stage without issuing
its copy (nothing is read or written out of bounds, nothing traps), with a
short poll limit so that every role gives up within milliseconds.  Afterwards
the status is read, and an ordinary call on the same context must be correct."""
import numpy as np
import pytest
import torch

from oracle import dk_field_oracle as F
from oracle import dk_oracle as O
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu


def spec_of(**kw):
    base = dict(workload="tiny", name="t", kind="conv", cin=64, cout=64, h=16, w=16, kh=3, kw=3, stride=1, pad=1,
                K=4, G=4, sigma_r=100.0)
    base.update(kw)
    return synth.LayerSpec(**base)


def arm(ctx, stage):
    dk.dk_set_option(ctx, dk.DK_OPT_SPIN_LIMIT, 1 << 12)
    dk.dk_set_option(ctx, dk.DK_OPT_TEST_WITHHOLD, stage)


def disarm(ctx):
    dk.dk_set_option(ctx, dk.DK_OPT_SPIN_LIMIT, 1 << 22)
    assert dk.dk_get_option(ctx, dk.DK_OPT_TEST_WITHHOLD) == -1      # the hook switched itself off


# single-CTA forward kernel, CTA-pair forward kernel (cout > 128), split-K forward (few tiles, long contraction)
FWD_CASES = [("single", spec_of(), 1), ("pair", spec_of(cout=256), 2), ("first_stage", spec_of(), 0)]


@pytest.mark.parametrize("name,spec,stage", FWD_CASES, ids=[c[0] for c in FWD_CASES])
def test_masked_linear_reports_a_wait_that_ran_out_and_recovers(name, spec, stage):
    ctx = dk.Context(0)
    try:
        d = synth.draw_layer(spec)
        p = dk.problem_from_spec(spec, tol=H.TAU)
        ctx.ensure_workspace(p)
        W = H.weights_to_dev(d["W"], dk.DK_NHWC)
        x, r = H.acts_to_dev(d["x"], dk.DK_NHWC), H.acts_to_dev(d["r"], dk.DK_NHWC)
        y = H.empty_acts(spec.batch, spec, "out", dk.DK_NHWC)
        v = dk.new_verdict()
        arm(ctx, stage)
        dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, None, v)      # returns: the kernel gave up
        vd = dk.read_verdict(v)
        assert vd["status"] == dk.DK_ERR_TIMEOUT and vd["ok"] == 0
        disarm(ctx)
        # the same context, an ordinary call: correct result, clean verdict
        dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, None, v)
        vd = dk.read_verdict(v)
        assert (vd["ok"], vd["n_flagged"], vd["status"]) == (1, 0, 0)
        plain = O.linear_plain(d["W"], d["x"], spec.stride, spec.pad)
        assert H.max_rel(H.acts_from_dev(y, dk.DK_NHWC), plain) < 1e-3
    finally:
        ctx.close()


@pytest.mark.parametrize("cout", [64, 256], ids=["single", "pair"])
def test_linear_fwd_and_wgrad_report_through_the_device_status(cout):
    spec = spec_of(cout=cout)
    ctx = dk.Context(0)
    try:
        d = synth.draw_layer(spec)
        p = dk.problem_from_spec(spec)
        ctx.ensure_workspace(p)
        E = spec.K + 2
        xbar32 = O.encode(d["x"], d["r"], d["C"]).astype(np.float32)
        W, xb = H.weights_to_dev(d["W"], dk.DK_NHWC), H.acts_to_dev(xbar32, dk.DK_NHWC)
        ybar = H.empty_acts(spec.G * E, spec, "out", dk.DK_NHWC)
        arm(ctx, 1)
        dk.dk_linear_fwd(ctx, p, W, xb, ybar)
        assert dk.dk_device_status(ctx) == dk.DK_ERR_TIMEOUT
        assert dk.dk_device_status(ctx) == 0                             # reading clears it
        disarm(ctx)
        dk.dk_linear_fwd(ctx, p, W, xb, ybar)
        assert dk.dk_device_status(ctx) == 0
        assert H.max_rel(H.acts_from_dev(ybar, dk.DK_NHWC), O.linear(d["W"], xbar32, spec.stride, spec.pad)) < 2e-5

        delta = H.acts_to_dev(d["delta"], dk.DK_NHWC)
        dW = H.empty_weights(spec, dk.DK_NHWC)
        scale = 1.0 / spec.batch
        arm(ctx, 2)
        dk.dk_linear_bwd_wgrad(ctx, p, delta, xb, E, d["C"], d["gamma"], scale, dW)
        assert dk.dk_device_status(ctx) == dk.DK_ERR_TIMEOUT
        disarm(ctx)
        dk.dk_linear_bwd_wgrad(ctx, p, delta, xb, E, d["C"], d["gamma"], scale, dW)
        assert dk.dk_device_status(ctx) == 0
        want = O.wgrad_plain(d["delta"], d["x"], scale, spec.kh, spec.kw, spec.stride, spec.pad)
        assert H.max_rel(H.weights_from_dev(dW, dk.DK_NHWC), want) < 1e-3
    finally:
        ctx.close()


def test_field_forward_kernel_reports_a_wait_that_ran_out_and_recovers():
    P, L = F.P_PAPER, F.L_PAPER
    spec = spec_of(cin=128, cout=128, K=2, G=2)
    ctx = dk.Context(0)
    try:
        d = synth.draw_field_layer(spec, P)
        p = dk.problem_from_spec(spec)
        ctx.ensure_workspace(p, field=True)
        E = spec.K + 2
        Wq, xq = F.quantize(d["W"], L, P), F.quantize(d["x"], L, P)
        xbar = F.field_encode(xq, d["rq"], d["Cq"], P)
        want = F.field_linear(Wq, xbar, P, spec.stride, spec.pad)

        def res(a):
            return torch.from_numpy(np.ascontiguousarray(a.transpose(0, 2, 3, 1)).astype(np.int32)).cuda()
        Wd, xd = res(Wq), res(xbar)
        ybar = torch.empty((spec.G * E, spec.hout, spec.wout, spec.cout), dtype=torch.int32, device="cuda")
        arm(ctx, 1)
        dk.dk_field_linear_fwd(ctx, p, P, Wd, xd, ybar)
        assert dk.dk_device_status(ctx) == dk.DK_ERR_TIMEOUT
        disarm(ctx)
        dk.dk_field_linear_fwd(ctx, p, P, Wd, xd, ybar)
        assert dk.dk_device_status(ctx) == 0
        assert np.array_equal(ybar.cpu().numpy().astype(np.int64).transpose(0, 3, 1, 2), want)
    finally:
        ctx.close()
