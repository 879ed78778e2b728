"""Detection floor of the floating-point integrity check (Section 4.4 compares
exactly in a finite field and has no floor; the floating-point rule flags
|rho| > tau * max(s_e, s_g)).  For one layer of each workload and every
encoding row: the smallest wrong value |delta| (in units of the rms of that
encoded output row) that is flagged at sampled output elements,

  * by the oracle's rule with the per-element scale s_e alone (the rule before
    the group term was introduced),
  * by the oracle's rule as it stands, max(s_e, s_g),
  * by the GPU, found by bisection on dk_fault.delta through dk_masked_linear.

The price of the group term is the ratio of the first two; the GPU must agree
with the oracle's rule as it stands.

    python -m pytest tests/test_gpu_detection_floor.py -m gpu -q -s

prints the table (the copy under profiles/ comes from this command)."""
import numpy as np
import pytest

from oracle import dk_oracle as O
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu

CASES = [("fc784:fc", synth.layers("fc784")[0]),
         ("vgg16_cifar:conv3_2", synth.layer("vgg16_cifar", "conv3_2").with_groups(2)),
         ("resnet18_224:layer3_3x3", synth.layer("resnet18_224", "layer3_3x3").with_groups(2)),
         ("mobilenetv2_pw:expand_64_384", synth.layer("mobilenetv2_pw", "expand_64_384").with_groups(2)),
         ("vgg16_224:conv5_1", synth.layer("vgg16_224", "conv5_1").with_groups(2))]
POSITIONS = 6


@pytest.fixture(scope="module")
def ctx():
    c = dk.Context(0)
    yield c
    c.close()


@pytest.fixture(scope="module", autouse=True)
def header():
    print(f"\n{'layer':32s} {'enc':>3s} {'|n_i|':>7s} {'s_e only (med/max)':>20s} {'max(s_e,s_g) (med/max)':>24s} "
          f"{'GPU (med/max)':>20s} {'price of group term':>20s}")
    yield


@pytest.mark.parametrize("name,spec", CASES, ids=[c[0] for c in CASES])
def test_detection_floor(ctx, name, spec):
    d = synth.draw_layer(spec)
    E, K = spec.K + 2, spec.K
    m = O.masked_forward(d["W"], d["x"], d["r"], d["C"], spec.stride, spec.pad, H.TAU)
    p = dk.problem_from_spec(spec, tol=H.TAU)
    ctx.ensure_workspace(p)
    W = H.weights_to_dev(d["W"], dk.DK_NHWC)
    x, r = H.acts_to_dev(d["x"], dk.DK_NHWC), H.acts_to_dev(d["r"], dk.DK_NHWC)
    y = H.empty_acts(spec.batch, spec, "out", dk.DK_NHWC)
    v = dk.new_verdict()
    rng = np.random.default_rng(83)
    for enc in range(E):
        se_only, both, gpu = [], [], []
        for _ in range(POSITIONS):
            g = int(rng.integers(0, spec.G))
            co, oh, ow = int(rng.integers(0, spec.cout)), int(rng.integers(0, spec.hout)), int(rng.integers(0, spec.wout))
            lidx = H.logical_out_index(spec, co, oh, ow)
            n = O.null_vector(d["C"][g])
            rows = m["ybar"][g * E:(g + 1) * E]
            rms = float(np.sqrt(np.mean(rows[enc] ** 2)))
            s_e = float(sum(abs(n[i]) * abs(rows[i][lidx]) for i in range(E)))
            s_max = float(m["scale"][(g,) + lidx])
            assert s_max >= s_e * (1 - 1e-12)
            se_only.append(H.TAU * s_e / abs(n[enc]) / rms)
            both.append(H.TAU * s_max / abs(n[enc]) / rms)
            lo, hi = 1e-3 * both[-1] * rms, 1e3 * both[-1] * rms
            flat = H.flat_out_index(spec, dk.DK_NHWC, co, oh, ow)
            for _ in range(22):
                mid = (lo * hi) ** 0.5
                dk.dk_masked_linear(ctx, p, W, x, r, d["C"], None, y, None, v, dk.dk_fault(g, enc, flat, mid))
                if dk.read_verdict(v)["n_flagged"] >= 1:
                    hi = mid
                else:
                    lo = mid
            gpu.append(hi / rms)
            # the GPU's floor is the oracle's, up to the GPU's own honest residual at that element
            assert 0.75 < gpu[-1] / both[-1] < 1.3, (name, enc, gpu[-1], both[-1])
        nmean = float(np.mean([abs(O.null_vector(d["C"][g])[enc]) for g in range(spec.G)]))
        print(f"{name:32s} {enc:3d} {nmean:7.3f} {np.median(se_only):9.2e} /{max(se_only):9.2e} "
              f"{np.median(both):11.2e} /{max(both):9.2e} {np.median(gpu):9.2e} /{max(gpu):9.2e} "
              f"{np.median(np.array(both) / np.array(se_only)):12.2f}x median")
