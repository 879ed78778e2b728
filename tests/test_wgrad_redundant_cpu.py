"""Pins of the oracle's redundant weight-gradient check: both equation sets
reproduce the plain gradient, a wrong element in either result is flagged
exactly there, a wrong encoded activation that only one set uses shows up as
the closed-form difference, and the second set's coefficients satisfy Eq. 5."""
import numpy as np
import pytest

from oracle import dk_oracle as O
from paper_2207_00083_b200 import synth


def tiny(kind, **kw):
    base = dict(workload="tiny", name="w", kind=kind, cin=5, cout=4, K=3, G=2, sigma_r=100.0)
    if kind == "conv":
        base.update(h=6, w=5, kh=3, kw=3, stride=1, pad=1)
    base.update(kw)
    return synth.LayerSpec(**base)


CASES = [tiny("fc"), tiny("conv"), tiny("conv", K=1, G=3), tiny("fc", K=4, G=1)]


@pytest.mark.parametrize("spec", CASES)
def test_both_equation_sets_give_the_plain_gradient(spec):
    d = synth.draw_layer(spec)
    xbar = O.encode(d["x"], d["r"], d["C"])
    scale = 1.0 / spec.batch
    r = O.wgrad_redundant(d["delta"], xbar, d["C"], d["gamma"], scale, spec.kh, spec.kw, spec.stride, spec.pad)
    plain = O.wgrad_plain(d["delta"], d["x"], scale, spec.kh, spec.kw, spec.stride, spec.pad)
    ref = float(np.max(np.abs(xbar))) * max(1.0, float(np.max(np.abs(plain))))
    assert np.max(np.abs(r["dW"] - plain)) <= 1e-9 * ref
    assert np.max(np.abs(r["dW_second"] - plain)) <= 1e-9 * ref
    assert not r["flags"].any()
    assert float(r["ratio"].max()) < 1e-6


@pytest.mark.parametrize("spec", CASES)
def test_second_set_satisfies_eq_5(spec):
    d = synth.draw_layer(spec)
    C2, g2 = O.second_equation_set(d["C"], d["gamma"])
    K = spec.K
    for g in range(spec.G):
        B = O.derive_B(C2[g], g2[g])
        A_T = C2[g][:K + 1]                       # C_sq = A^T
        res = B.T @ np.diag(g2[g]) @ A_T          # B^T Gamma A^T must be [I_K | 0]
        want = np.concatenate([np.eye(K), np.zeros((K, 1))], axis=1)
        assert np.max(np.abs(res - want)) < 1e-10
        # rows of the second set are rows 1..K+1 of the first
        assert np.array_equal(C2[g][:K + 1], d["C"][g][1:K + 2])


@pytest.mark.parametrize("which", [0, 1])
def test_wrong_result_element_is_flagged_exactly_there(which):
    spec = tiny("conv")
    d = synth.draw_layer(spec)
    xbar = O.encode(d["x"], d["r"], d["C"])
    scale = 1.0 / spec.batch
    clean = O.wgrad_redundant(d["delta"], xbar, d["C"], d["gamma"], scale, spec.kh, spec.kw, spec.stride, spec.pad)
    idx = (spec.cout - 1, 2, 0, 1)
    bad = O.wgrad_redundant(d["delta"], xbar, d["C"], d["gamma"], scale, spec.kh, spec.kw, spec.stride, spec.pad,
                            fault=(which, idx, 0.5 * clean["rms"]))
    assert bad["flags"].sum() == 1 and bad["flags"][idx]
    # the normaliser is the rms of the first result as it came back (fault included)
    assert bad["ratio"][idx] == pytest.approx(0.5 * clean["rms"] / bad["rms"], rel=1e-6)


def test_wrong_encoding_used_by_one_set_only_gives_the_closed_form_difference():
    """Encoding 0 enters the first set only: corrupting one of its elements by D shifts the first
    result by scale * gamma_0 * <delta_bar_0, D e> and leaves the second untouched."""
    spec = tiny("fc", K=2, G=1)
    d = synth.draw_layer(spec)
    xbar = O.encode(d["x"], d["r"], d["C"])
    scale = 0.5
    clean = O.wgrad_redundant(d["delta"], xbar, d["C"], d["gamma"], scale)
    xbad = xbar.copy()
    D, e = 3.0, 2
    xbad[0, e] += D
    bad = O.wgrad_redundant(d["delta"], xbad, d["C"], d["gamma"], scale)
    assert np.allclose(bad["dW_second"], clean["dW_second"], rtol=0, atol=0)
    B = O.derive_B(d["C"][0], d["gamma"][0])
    dbar0 = sum(B[0, i] * d["delta"][i].astype(np.float64) for i in range(spec.K))
    want = np.zeros_like(clean["dW"])
    want[:, e] = scale * d["gamma"][0, 0] * dbar0 * D
    assert np.max(np.abs((bad["dW"] - clean["dW"]) - want)) <= 1e-9 * np.max(np.abs(want))
    assert bad["flags"][:, e].all() and not np.delete(bad["flags"], e, axis=1).any()
