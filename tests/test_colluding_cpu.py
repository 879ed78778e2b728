"""Pins of the oracle's colluding-accelerator functions (the paper's scheme with
M noise vectors and S = K + M encodings): round trip against the plain
definition, the rank condition on A2, the weight-gradient identity, the M = 1
case against Eq. 1, and the relabelling under which the library's interface
(K_lib = K + M - 1 "inputs", the last M - 1 of them noise) is the same scheme."""
import dataclasses

import numpy as np
import pytest

from oracle import dk_oracle as O
from paper_2207_00083_b200 import synth


def spec_for(kind, K, M, **kw):
    base = dict(workload="tiny", name="c", kind=kind, cin=6, cout=5, K=K + M - 1, G=2, sigma_r=100.0)
    if kind == "conv":
        base.update(h=6, w=5, kh=3, kw=3, stride=1, pad=1)
    base.update(kw)
    return synth.LayerSpec(**base)


CASES = [("fc", 2, 3), ("conv", 3, 2), ("conv", 1, 4), ("fc", 4, 1)]


@pytest.mark.parametrize("kind,K,M", CASES)
def test_round_trip_reproduces_the_plain_result(kind, K, M):
    spec = spec_for(kind, K, M)
    d = synth.draw_colluding(spec, K, M)
    for g in range(spec.G):
        xbar = O.encode_colluding(d["x_private"][g], d["R"][g], d["A1"][g], d["A2"][g])
        ybar = O.linear(d["W"], xbar, spec.stride, spec.pad)
        y, z = O.decode_colluding(ybar, d["A1"][g], d["A2"][g])
        want_y = O.linear_plain(d["W"], d["x_private"][g], spec.stride, spec.pad)
        want_z = O.linear(d["W"], d["R"][g], spec.stride, spec.pad)
        assert np.max(np.abs(y - want_y)) <= 1e-9 * max(1.0, np.max(np.abs(want_z)))
        assert np.max(np.abs(z - want_z)) <= 1e-9 * np.max(np.abs(want_z))


@pytest.mark.parametrize("kind,K,M", CASES)
def test_library_interface_expresses_the_same_scheme(kind, K, M):
    """encode() on [x_private, r_1..r_{M-1}] with noise r_M and C = [A^T; redundant row]
    gives the S encodings of encode_colluding, and its decode gives the same y."""
    spec = spec_for(kind, K, M)
    d = synth.draw_colluding(spec, K, M)
    S, E = K + M, spec.K + 2
    xbar_lib = O.encode(d["x"], d["r"], d["C"])
    m = O.masked_forward(d["W"], d["x"], d["r"], d["C"], spec.stride, spec.pad)
    for g in range(spec.G):
        want = O.encode_colluding(d["x_private"][g], d["R"][g], d["A1"][g], d["A2"][g])
        got = xbar_lib[g * E:g * E + S]
        assert np.max(np.abs(got - want)) <= 1e-10 * np.max(np.abs(want))
        y_lib = m["y"][g * spec.K:g * spec.K + K]
        want_y = O.linear_plain(d["W"], d["x_private"][g], spec.stride, spec.pad)
        assert np.max(np.abs(y_lib - want_y)) <= 1e-8 * max(1.0, np.max(np.abs(m["ybar"])))
    assert m["flags"].sum() == 0


def test_m_equal_one_is_eq_1():
    spec = spec_for("fc", 3, 1)
    d = synth.draw_colluding(spec, 3, 1)
    E = spec.K + 2
    lib = O.encode(d["x"], d["r"], d["C"])
    for g in range(spec.G):
        got = O.encode_colluding(d["x_private"][g], d["R"][g], d["A1"][g], d["A2"][g])
        assert np.allclose(got, lib[g * E:g * E + spec.K + 1], rtol=1e-12, atol=0)


def test_rank_condition_on_the_noise_block():
    spec = spec_for("fc", 2, 3)
    d = synth.draw_colluding(spec, 2, 3)
    for g in range(spec.G):
        assert O.colluding_subsets_full_rank(d["A2"][g])
    bad = d["A2"][0].copy()
    bad[:, 1] = 2.5 * bad[:, 0]          # two encodings whose noise parts are proportional
    assert not O.colluding_subsets_full_rank(bad)
    # by hand, M = 1: a zero noise coefficient leaves that encoding unmasked
    assert O.colluding_subsets_full_rank(np.array([[1.0, -2.0, 0.5]]))
    assert not O.colluding_subsets_full_rank(np.array([[1.0, 0.0, 0.5]]))


@pytest.mark.parametrize("kind,K,M", CASES)
def test_weight_gradient_identity(kind, K, M):
    spec = spec_for(kind, K, M)
    d = synth.draw_colluding(spec, K, M)
    S, E = K + M, spec.K + 2
    scale = 0.25
    xbar_lib = O.encode(d["x"], d["r"], d["C"])
    total = None
    for g in range(spec.G):
        xbar = O.encode_colluding(d["x_private"][g], d["R"][g], d["A1"][g], d["A2"][g])
        part = O.wgrad_colluding(d["delta_private"][g], xbar, d["A1"][g], d["A2"][g], d["gamma"][g], scale,
                                 spec.kh, spec.kw, spec.stride, spec.pad)
        total = part if total is None else total + part
    xp = d["x_private"].reshape((spec.G * K,) + d["x_private"].shape[2:])
    dp = d["delta_private"].reshape((spec.G * K,) + d["delta_private"].shape[2:])
    plain = O.wgrad_plain(dp, xp, scale, spec.kh, spec.kw, spec.stride, spec.pad)
    ref = max(1.0, float(np.max(np.abs(xbar_lib))))
    assert np.max(np.abs(total - plain)) <= 1e-9 * ref * max(1.0, float(np.max(np.abs(plain))))
    # the library's interface: deltas of the noise rows are zero
    lib = O.wgrad_masked(d["delta"], xbar_lib, d["C"], d["gamma"], scale, spec.kh, spec.kw, spec.stride,
                         spec.pad, xbar_rows_per_group=E)
    assert np.max(np.abs(lib - plain)) <= 1e-9 * ref * max(1.0, float(np.max(np.abs(plain))))
