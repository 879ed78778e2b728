"""Measured-error table of the GPU arithmetic modes against the fp64 oracle.

    python -m tests.error_table

For every small parity case: max-norm relative error of y_bar (dk_linear_fwd on
identical fp32 encodings) and of the decoded y (dk_masked_linear against the
plain definition), the honest max_ratio of the integrity check and the error of dW
(dk_linear_bwd_wgrad on fp32 encodings against the plain definition), for the
tensor-core 3xTF32 mode, the fp32 SIMT mode and the fp64 mode.  Reporting aid
for the choice of arithmetic; the pass/fail bars live in the test files."""
import numpy as np

from oracle import dk_oracle as O
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth
from tests import harness as H
from tests.test_gpu_parity import CASES


def main():
    ctx = dk.Context(0)
    extra = [("vgg_cifar_conv4_2_G4", synth.layer("vgg16_cifar", "conv4_2").with_groups(4)),
             ("vgg_cifar_conv1_2_G2", synth.layer("vgg16_cifar", "conv1_2").with_groups(2)),
             ("mbv2_expand_160_960_G2", synth.layer("mobilenetv2_pw", "expand_160_960").with_groups(2))]
    print(f"{'case':28s} {'K':>2s} {'sigma':>6s} {'kc':>6s} {'mode':>6s} {'ybar':>9s} {'y':>9s} {'maxratio':>9s} "
          f"{'dW':>9s}")
    for name, spec in CASES + extra:
        d = synth.draw_layer(spec)
        K, E = spec.K, spec.K + 2
        xbar32 = O.encode(d["x"], d["r"], d["C"]).astype(np.float32)
        want_yb = O.linear(d["W"], xbar32, spec.stride, spec.pad)
        plain = O.linear_plain(d["W"], d["x"], spec.stride, spec.pad)
        for prec, pn in ((dk.DK_TF32X3, "tf32x3"), (dk.DK_FP32_SIMT, "fp32"), (dk.DK_FP64_SIMT, "fp64")):
            p = dk.problem_from_spec(spec, precision=prec, tol=1e-4)
            ctx.ensure_workspace(p)
            W = H.weights_to_dev(d["W"], 0)
            ybar = H.empty_acts(spec.G * E, spec, "out", 0)
            dk.dk_linear_fwd(ctx, p, W, H.acts_to_dev(xbar32, 0), ybar)
            e1 = H.max_rel(H.acts_from_dev(ybar, 0), want_yb)
            y = H.empty_acts(spec.G * K, spec, "out", 0)
            v = dk.new_verdict()
            dk.dk_masked_linear(ctx, p, W, H.acts_to_dev(d["x"], 0), H.acts_to_dev(d["r"], 0), d["C"], None, y,
                                None, v)
            e2 = H.max_rel(H.acts_from_dev(y, 0), plain)
            vd = dk.read_verdict(v)
            dW = H.empty_weights(spec, 0)
            scale = 1.0 / spec.batch
            dk.dk_linear_bwd_wgrad(ctx, p, H.acts_to_dev(d["delta"], 0), H.acts_to_dev(xbar32, 0), E, d["C"],
                                   d["gamma"], scale, dW)
            want_dw = O.wgrad_plain(d["delta"], d["x"], scale, spec.kh, spec.kw, spec.stride, spec.pad)
            e3 = H.max_rel(H.weights_from_dev(dW, 0), want_dw)
            print(f"{name:28s} {K:2d} {spec.sigma_r:6.0f} {spec.kc:6d} {pn:>6s} {e1:9.2e} {e2:9.2e} "
                  f"{vd['max_ratio']:9.2e} {e3:9.2e} ok={vd['ok']}")
    ctx.close()


if __name__ == "__main__":
    main()
