"""Measured error of every arithmetic mode of the GPU path against the fp64
oracle, one row per (case, mode): max-norm relative error of y_bar
(dk_linear_fwd on identical fp32 encodings), of the decoded y (dk_masked_linear
against the plain definition <W, x>), the honest max |rho|/s_g of the integrity
check, and the error of dW (dk_linear_bwd_wgrad against the plain definition).

    python -m pytest tests/test_gpu_error_table.py -m gpu -q -s

prints the table (the copy under profiles/ comes from this command).  The
bars asserted here are the ones the choice of arithmetic rests on: 1e-3 on y
and dW wherever a mode is offered for that noise level."""
import os

import numpy as np
import pytest

from oracle import dk_oracle as O
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth
from tests import harness as H
from tests.test_gpu_parity import CASES

pytestmark = pytest.mark.gpu

EXTRA = [("vgg_cifar_conv4_2_G4", synth.layer("vgg16_cifar", "conv4_2").with_groups(4)),
         ("vgg_cifar_conv1_2_G2", synth.layer("vgg16_cifar", "conv1_2").with_groups(2)),
         ("mbv2_expand_160_960_G2", synth.layer("mobilenetv2_pw", "expand_160_960").with_groups(2))]
ALL = CASES + EXTRA
MODES = [(dk.DK_TF32X3, "tf32x3"), (dk.DK_TF32X2_WUNSPLIT, "tf32x2w"), (dk.DK_FP32_SIMT, "fp32"), (dk.DK_FP64_SIMT, "fp64")]


@pytest.fixture(scope="module")
def ctx():
    """The chunk lengths of the tensor-memory accumulation change the arithmetic; DK_TEST_TC_CHUNK / DK_TEST_WG_CHUNK
    in the environment of this test set the context's options for a sweep (profiles/error_vs_tmem_chunk_*)."""
    c = dk.Context(0)
    if os.environ.get("DK_TEST_TC_CHUNK"):
        dk.dk_set_option(c, dk.DK_OPT_TC_CHUNK, int(os.environ["DK_TEST_TC_CHUNK"]))
    if os.environ.get("DK_TEST_WG_CHUNK"):
        dk.dk_set_option(c, dk.DK_OPT_WG_CHUNK, int(os.environ["DK_TEST_WG_CHUNK"]))
    yield c
    c.close()


@pytest.fixture(scope="module", autouse=True)
def header():
    print(f"\n{'case':28s} {'K':>2s} {'sigma':>6s} {'kc':>6s} {'mode':>8s} {'ybar':>9s} {'y':>9s} {'maxratio':>9s} "
          f"{'dW':>9s}")
    yield


def measure(ctx, spec, d, prec):
    K, E = spec.K, spec.K + 2
    xbar32 = O.encode(d["x"], d["r"], d["C"]).astype(np.float32)
    want_yb = O.linear(d["W"], xbar32, spec.stride, spec.pad)
    plain = O.linear_plain(d["W"], d["x"], spec.stride, spec.pad)
    p = dk.problem_from_spec(spec, precision=prec, tol=1e-4)
    ctx.ensure_workspace(p)
    W = H.weights_to_dev(d["W"], 0)
    ybar = H.empty_acts(spec.G * E, spec, "out", 0)
    dk.dk_linear_fwd(ctx, p, W, H.acts_to_dev(xbar32, 0), ybar)
    e_ybar = H.max_rel(H.acts_from_dev(ybar, 0), want_yb)
    y = H.empty_acts(spec.G * K, spec, "out", 0)
    v = dk.new_verdict()
    dk.dk_masked_linear(ctx, p, W, H.acts_to_dev(d["x"], 0), H.acts_to_dev(d["r"], 0), d["C"], None, y, None, v)
    e_y = H.max_rel(H.acts_from_dev(y, 0), plain)
    vd = dk.read_verdict(v)
    dW = H.empty_weights(spec, 0)
    scale = 1.0 / spec.batch
    dk.dk_linear_bwd_wgrad(ctx, p, H.acts_to_dev(d["delta"], 0), H.acts_to_dev(xbar32, 0), E, d["C"], d["gamma"],
                           scale, dW)
    want_dw = O.wgrad_plain(d["delta"], d["x"], scale, spec.kh, spec.kw, spec.stride, spec.pad)
    e_dw = H.max_rel(H.weights_from_dev(dW, 0), want_dw)
    return e_ybar, e_y, vd, e_dw


@pytest.mark.parametrize("prec,pn", MODES, ids=[m[1] for m in MODES])
@pytest.mark.parametrize("name,spec", ALL, ids=[c[0] for c in ALL])
def test_error_of_mode(ctx, name, spec, prec, pn):
    d = synth.draw_layer(spec)
    e_ybar, e_y, vd, e_dw = measure(ctx, spec, d, prec)
    print(f"{name:28s} {spec.K:2d} {spec.sigma_r:6.0f} {spec.kc:6d} {pn:>8s} {e_ybar:9.2e} {e_y:9.2e} "
          f"{vd['max_ratio']:9.2e} {e_dw:9.2e} ok={vd['ok']}")
    assert vd["status"] == 0
    if pn == "fp64":
        assert vd["ok"] == 1 and e_y < 1e-6 and e_dw < 1e-3
    elif pn == "tf32x2w" and spec.sigma_r <= 100.0:
        # W as one TF32 term: the bar this opt-in mode is offered under (half the tolerance)
        assert vd["ok"] == 1 and e_y < 5e-4 and e_dw < 1e-3
    elif spec.sigma_r <= 100.0:
        assert vd["ok"] == 1 and e_y < 1e-3 and e_dw < 1e-3
    else:
        # noise 1000x the inputs: fp32 accumulators lose 2^-24 of a running sum that is ~1000x the signal, the
        # decoder multiplies that by its gain; these rows are why that noise level runs in the fp64 mode.
        # Recorded, not held to the bar.
        assert np.isfinite(e_y) and e_y < 5e-2
