"""Pins for the fp64 oracle: everything here runs on the CPU and checks the
oracle against things that are fixed by the paper and by mathematics, never
against itself and never against the CUDA path."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import dk_oracle as O
from paper_2207_00083_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rel(a, b):
    return float(np.max(np.abs(np.asarray(a) - np.asarray(b))) / max(np.max(np.abs(b)), 1e-300))


def tiny_conv_spec(K=2, G=2, cin=3, cout=4, hw=5, k=3, s=1, p=1, sigma=100.0):
    return synth.LayerSpec("tiny", "t", "conv", cin, cout, hw, hw, k, k, s, p, K=K, G=G, sigma_r=sigma)


def tiny_fc_spec(K=2, G=2, cin=7, cout=5, sigma=100.0):
    return synth.LayerSpec("tiny", "t", "fc", cin, cout, K=K, G=G, sigma_r=sigma)


# ---------------------------------------------------------------------------
# small linear algebra
# ---------------------------------------------------------------------------
def test_invert_is_two_sided_inverse_and_pivots():
    rng = np.random.default_rng(1)
    for n in (1, 2, 3, 5, 9):
        M = rng.standard_normal((n, n))
        Mi = O.invert(M)
        assert np.allclose(M @ Mi, np.eye(n), atol=1e-10)
        assert np.allclose(Mi @ M, np.eye(n), atol=1e-10)
    # zero on the diagonal: only works with row exchanges
    M = np.array([[0.0, 2.0], [3.0, 1.0]])
    assert np.allclose(O.invert(M), np.array([[-1 / 6, 1 / 3], [1 / 2, 0.0]]))
    with pytest.raises(ZeroDivisionError):
        O.invert(np.array([[1.0, 2.0], [2.0, 4.0]]))


def test_null_vector_annihilates_C():
    rng = np.random.default_rng(2)
    for K in (1, 2, 4, 8):
        C = synth.draw_coefficients(rng, K, 1)[0]
        n = O.null_vector(C)
        assert n[-1] == 1.0
        assert np.max(np.abs(n @ C.astype(np.float64))) < 1e-12


# ---------------------------------------------------------------------------
# encode (Eq. 1)
# ---------------------------------------------------------------------------
def test_encode_identity_coefficients_pass_inputs_through():
    K, G = 3, 2
    rng = np.random.default_rng(3)
    x = rng.standard_normal((G * K, 2, 3, 3))
    r = rng.standard_normal((G, 2, 3, 3))
    C = np.zeros((G, K + 2, K + 1))
    C[:, :K + 1] = np.eye(K + 1)
    C[:, K + 1] = 1.0                       # redundant row: plain sum
    xb = O.encode(x, r, C)
    for g in range(G):
        for k in range(K):
            assert np.array_equal(xb[g * (K + 2) + k], x[g * K + k])
        assert np.array_equal(xb[g * (K + 2) + K], r[g])
        assert np.allclose(xb[g * (K + 2) + K + 1], x[g * K:(g + 1) * K].sum(0) + r[g])


def test_encode_K1_by_hand():
    # one private input plus noise -> x0 = a x + c r, x1 = b x + d r, x2 = e x + f r
    x = np.array([[2.0, -1.0]])
    r = np.array([[10.0, 4.0]])
    C = np.array([[[3.0, 0.5], [-2.0, 1.5], [1.0, -1.0]]])
    xb = O.encode(x, r, C)
    assert np.array_equal(xb, np.array([[11.0, -1.0], [11.0, 8.0], [-8.0, -5.0]]))


def test_encode_exact_rational_bruteforce():
    K, G, n = 2, 2, 4
    rng = np.random.default_rng(4)
    x = rng.integers(-5, 6, (G * K, n)).astype(np.float64)
    r = rng.integers(-50, 51, (G, n)).astype(np.float64)
    C = rng.integers(-4, 5, (G, K + 2, K + 1)).astype(np.float64)
    xb = O.encode(x, r, C)
    for g, i, e in itertools.product(range(G), range(K + 2), range(n)):
        want = sum(Fraction(int(C[g, i, k])) * int(x[g * K + k, e]) for k in range(K))
        want += Fraction(int(C[g, i, K])) * int(r[g, e])
        assert Fraction(xb[g * (K + 2) + i, e]) == want


# ---------------------------------------------------------------------------
# the bilinear operation
# ---------------------------------------------------------------------------
def brute_conv(W, x, s, p):
    n, cin, h, w = x.shape
    cout, _, kh, kw = W.shape
    ho, wo = (h + 2 * p - kh) // s + 1, (w + 2 * p - kw) // s + 1
    y = np.zeros((n, cout, ho, wo))
    for b, o, a, q, c, u, v in itertools.product(range(n), range(cout), range(ho), range(wo),
                                                 range(cin), range(kh), range(kw)):
        ih, iw = a * s + u - p, q * s + v - p
        if 0 <= ih < h and 0 <= iw < w:
            y[b, o, a, q] += W[o, c, u, v] * x[b, c, ih, iw]
    return y


@pytest.mark.parametrize("k,s,p,hw", [(3, 1, 1, 5), (3, 2, 1, 6), (1, 2, 0, 6), (7, 2, 3, 9), (1, 1, 0, 4)])
def test_linear_conv_matches_bruteforce_loops(k, s, p, hw):
    rng = np.random.default_rng(5)
    x = rng.standard_normal((2, 3, hw, hw))
    W = rng.standard_normal((4, 3, k, k))
    assert rel(O.linear(W, x, s, p), brute_conv(W, x, s, p)) < 1e-13


@pytest.mark.parametrize("k,s,p,hw,cin,cout", [(3, 1, 1, 16, 8, 12), (3, 2, 1, 15, 5, 7),
                                               (7, 2, 3, 32, 3, 8), (1, 2, 0, 14, 16, 8)])
def test_linear_conv_matches_library_float64(k, s, p, hw, cin, cout):
    rng = np.random.default_rng(6)
    x = rng.standard_normal((3, cin, hw, hw))
    W = rng.standard_normal((cout, cin, k, k))
    ref = torch.nn.functional.conv2d(torch.from_numpy(x), torch.from_numpy(W), stride=s, padding=p).numpy()
    got = O.linear(W, x, s, p)
    assert got.shape == ref.shape
    assert rel(got, ref) < 1e-12
    # single-element evaluation agrees with the full tensor
    for (b, o, a, q) in [(0, 0, 0, 0), (2, cout - 1, ref.shape[2] - 1, ref.shape[3] - 1), (1, 1, 1, 0)]:
        assert abs(O.linear_at(W, x[b], o, a, q, s, p) - ref[b, o, a, q]) < 1e-10


def test_linear_fc_is_matrix_vector_product():
    rng = np.random.default_rng(7)
    x = rng.standard_normal((3, 6))
    W = rng.standard_normal((4, 6))
    y = O.linear(W, x)
    for b, o in itertools.product(range(3), range(4)):
        assert abs(y[b, o] - sum(W[o, c] * x[b, c] for c in range(6))) < 1e-13
    assert abs(O.linear_at(W, x[1], 2, 0, 0) - y[1, 2]) < 1e-13


# ---------------------------------------------------------------------------
# decode (Eq. 2): decode(<W, encode(X)>) = <W, X>
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("K,sigma", [(1, 100.0), (2, 100.0), (4, 100.0), (8, 1000.0)])
def test_decode_roundtrip_equals_plain_conv(K, sigma):
    spec = tiny_conv_spec(K=K, G=2, sigma=sigma)
    d = synth.draw_layer(spec)
    m = O.masked_forward(d["W"], d["x"], d["r"], d["C"], spec.stride, spec.pad)
    plain = O.linear_plain(d["W"], d["x"], spec.stride, spec.pad)
    assert rel(m["y"], plain) < 1e-9
    # the dropped unknown is <W, r>
    assert rel(m["z"], O.linear(d["W"], d["r"], spec.stride, spec.pad)) < 1e-9


def test_decode_roundtrip_fc_config1_shape():
    spec = synth.layers("fc784")[0]
    d = synth.draw_layer(spec)
    m = O.masked_forward(d["W"], d["x"], d["r"], d["C"])
    assert m["ybar"].shape == (4, 512)
    assert rel(m["y"], d["x"].astype(np.float64) @ d["W"].astype(np.float64).T) < 1e-10


def test_decode_K1_closed_form():
    # y_bar0 = a y + c z, y_bar1 = b y + d z  =>  y = (d y_bar0 - c y_bar1)/(ad - bc)
    a, c, b, d = 1.5, -0.7, 0.4, 2.0
    C = np.array([[[a, c], [b, d], [0.3, 0.9]]])
    ybar = np.array([[2.0, -3.0], [1.0, 5.0], [0.0, 0.0]])
    y, z = O.decode(ybar, C)
    det = a * d - b * c
    assert np.allclose(y[0], (d * ybar[0] - c * ybar[1]) / det, rtol=1e-14)
    assert np.allclose(z[0], (-b * ybar[0] + a * ybar[1]) / det, rtol=1e-14)


def test_decode_exact_rational_tiny_fc():
    """Whole masked forward in exact rational arithmetic on integer data."""
    K, n_in, n_out = 2, 3, 2
    rng = np.random.default_rng(8)
    x = rng.integers(-3, 4, (K, n_in))
    r = rng.integers(-40, 41, (1, n_in))
    W = rng.integers(-3, 4, (n_out, n_in))
    C = np.array([[[1, 2, 1], [0, 1, 3], [2, -1, 1], [1, 1, -2]]])
    got = O.masked_forward(W.astype(float), x.astype(float), r.astype(float), C.astype(float))
    src = [[Fraction(int(v)) for v in row] for row in list(x) + list(r)]
    xbar = [[sum(Fraction(int(C[0, i, k])) * src[k][e] for k in range(K + 1)) for e in range(n_in)]
            for i in range(K + 2)]
    ybar = [[sum(Fraction(int(W[o, e])) * xbar[i][e] for e in range(n_in)) for o in range(n_out)]
            for i in range(K + 2)]
    for i, o in itertools.product(range(K + 2), range(n_out)):
        assert abs(got["ybar"][i, o] - float(ybar[i][o])) < 1e-9
    for k, o in itertools.product(range(K), range(n_out)):
        want = sum(int(W[o, e]) * int(x[k, e]) for e in range(n_in))
        assert abs(got["y"][k, o] - want) < 1e-9


def test_pins_catch_a_transposed_coefficient_matrix():
    """Plant a mistake on the CPU: decoding with C_sq^T must break the round trip."""
    spec = tiny_fc_spec(K=3, G=1)
    d = synth.draw_layer(spec)
    xbar = O.encode(d["x"], d["r"], d["C"])
    ybar = O.linear(d["W"], xbar)
    Cbad = d["C"].copy()
    Cbad[0, :4] = d["C"][0, :4].T
    ybad, _ = O.decode(ybar, Cbad)
    assert rel(ybad, O.linear_plain(d["W"], d["x"])) > 1e-2


# ---------------------------------------------------------------------------
# verify (Section 4.4)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("K", [1, 2, 4, 8])
def test_verify_clean_run_has_zero_residual(K):
    spec = tiny_conv_spec(K=K, G=2, sigma=1000.0)
    d = synth.draw_layer(spec)
    m = O.masked_forward(d["W"], d["x"], d["r"], d["C"], spec.stride, spec.pad)
    assert m["ratio"].max() < 1e-10
    assert not m["flags"].any()
    v = O.verdict(m["flags"], m["ratio_group"])
    assert v == {"ok": 1, "n_flagged": 0, "first_index": -1, "max_ratio": v["max_ratio"]}


@pytest.mark.parametrize("enc", [0, 1, 2, 3, 4, 5])
def test_verify_single_fault_changes_one_residual_by_n_times_delta(enc):
    K = 4
    spec = tiny_conv_spec(K=K, G=2)
    d = synth.draw_layer(spec)
    g, idx, dlt = 1, (2, 3, 1), 0.75
    clean = O.masked_forward(d["W"], d["x"], d["r"], d["C"], spec.stride, spec.pad)
    bad = O.masked_forward(d["W"], d["x"], d["r"], d["C"], spec.stride, spec.pad,
                           fault=(g * (K + 2) + enc, idx, dlt))
    n = O.null_vector(d["C"][g])
    diff = bad["rho"] - clean["rho"]
    assert abs(diff[(g,) + idx] - n[enc] * dlt) < 1e-9
    diff[(g,) + idx] = 0.0
    assert np.max(np.abs(diff)) < 1e-9
    assert bad["flags"].sum() == 1 and bad["flags"][(g,) + idx]
    v = O.verdict(bad["flags"], bad["ratio"])
    assert v["ok"] == 0 and v["n_flagged"] == 1
    assert v["first_index"] == np.ravel_multi_index((g,) + idx, bad["flags"].shape)


def test_verify_equals_disagreement_between_equation_subsets():
    """Decoding from any two (K+1)-subsets of the K+2 equations differs by a
    multiple of the residual; on a clean run all subsets agree."""
    K = 3
    spec = tiny_fc_spec(K=K, G=1)
    d = synth.draw_layer(spec)
    C = d["C"][0].astype(np.float64)
    for fault in (None, (2, (3,), 0.5)):
        m = O.masked_forward(d["W"], d["x"], d["r"], d["C"], fault=fault)
        sols = []
        for drop in range(K + 2):
            rows = [i for i in range(K + 2) if i != drop]
            sols.append(np.linalg.solve(C[rows], m["ybar"][rows]))
        for a, b in itertools.combinations(range(K + 2), 2):
            dif = sols[a] - sols[b]                     # [K+1, n_out]
            if fault is None:
                assert np.max(np.abs(dif)) < 1e-8
            else:
                # rank one: every column is proportional to rho at that element
                nz = np.abs(m["rho"][0]) > 1e-6
                assert nz.sum() == 1
                assert np.max(np.abs(dif[:, ~nz])) < 1e-8
                assert np.max(np.abs(dif[:, nz])) > 1e-3


def test_verify_threshold_is_relative_to_noise_scale():
    K = 2
    spec = tiny_fc_spec(K=K, G=1)
    d = synth.draw_layer(spec)
    m = O.masked_forward(d["W"], d["x"], d["r"], d["C"])
    n = O.null_vector(d["C"][0])
    s = m["scale"][0, 1]
    # a fault 10x below the floor passes, one 10x above is flagged
    for factor, want in ((0.1, 0), (10.0, 1)):
        dlt = factor * 1e-4 * s / abs(n[0])
        bad = O.masked_forward(d["W"], d["x"], d["r"], d["C"], fault=(0, (1,), dlt))
        assert int(bad["flags"].sum()) == want


def test_verify_does_not_flag_rounding_where_all_encodings_vanish():
    """Where <W, r> and <W, x> vanish (a zero filter row) every y_bar is ~0 at
    once; a rounding-sized residual there must not raise the flag, while the
    same residual scaled up to the group's noise level must."""
    spec = tiny_fc_spec(K=2, G=1, cin=32, cout=16)
    d = synth.draw_layer(spec)
    W = d["W"].copy()
    W[3] = 0.0
    clean = O.masked_forward(W, d["x"], d["r"], d["C"])
    typical = float(np.sqrt(np.mean(clean["ybar"] ** 2)))
    tiny_err = O.masked_forward(W, d["x"], d["r"], d["C"], fault=(1, (3,), 1e-7 * typical))
    assert not tiny_err["flags"].any()
    big_err = O.masked_forward(W, d["x"], d["r"], d["C"], fault=(1, (3,), 1e-1 * typical))
    assert big_err["flags"].sum() == 1 and big_err["flags"][0, 3]


def test_verify_flags_an_infinity_from_the_accelerator():
    spec = tiny_fc_spec(K=2, G=1)
    d = synth.draw_layer(spec)
    bad = O.masked_forward(d["W"], d["x"], d["r"], d["C"], fault=(0, (1,), float("inf")))
    assert bad["flags"].sum() == 1 and bad["flags"][0, 1]


def test_verify_flags_a_nan_from_the_accelerator():
    spec = tiny_fc_spec(K=2, G=1)
    d = synth.draw_layer(spec)
    bad = O.masked_forward(d["W"], d["x"], d["r"], d["C"], fault=(3, (2,), float("nan")))
    assert bad["flags"].sum() == 1 and bad["flags"][0, 2]


# ---------------------------------------------------------------------------
# wgrad (Eq. 4-6)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("K", [1, 2, 4, 8])
def test_B_satisfies_eq5(K):
    rng = np.random.default_rng(9)
    C = synth.draw_coefficients(rng, K, 1)[0]
    gamma = synth.draw_gamma(rng, K, 1)[0]
    B = O.derive_B(C, gamma)
    A = C[:K + 1].astype(np.float64).T
    lhs = B.T @ np.diag(gamma.astype(np.float64)) @ A.T
    want = np.concatenate([np.eye(K), np.zeros((K, 1))], axis=1)
    assert np.max(np.abs(lhs - want)) < 1e-12


def brute_wgrad_conv(delta, x, k, s, p):
    n, cout, ho, wo = delta.shape
    cin, h, w = x.shape[1:]
    dW = np.zeros((cout, cin, k, k))
    for b, o, c, u, v, a, q in itertools.product(range(n), range(cout), range(cin), range(k), range(k),
                                                 range(ho), range(wo)):
        ih, iw = a * s + u - p, q * s + v - p
        if 0 <= ih < h and 0 <= iw < w:
            dW[o, c, u, v] += delta[b, o, a, q] * x[b, c, ih, iw]
    return dW


@pytest.mark.parametrize("k,s,p,hw", [(3, 1, 1, 5), (3, 2, 1, 6), (1, 1, 0, 4)])
def test_wgrad_plain_matches_bruteforce(k, s, p, hw):
    rng = np.random.default_rng(10)
    x = rng.standard_normal((2, 3, hw, hw))
    ho = (hw + 2 * p - k) // s + 1
    delta = rng.standard_normal((2, 4, ho, ho))
    got = O.wgrad_plain(delta, x, 0.5, k, k, s, p)
    assert rel(got, 0.5 * brute_wgrad_conv(delta, x, k, s, p)) < 1e-13
    assert abs(O.wgrad_plain_at(delta, x, 0.5, 3, 2, k - 1, 0, s, p) - got[3, 2, k - 1, 0]) < 1e-12


@pytest.mark.parametrize("k,s,p,hw", [(3, 1, 1, 8), (3, 2, 1, 9), (7, 2, 3, 16), (1, 2, 0, 8)])
def test_wgrad_plain_matches_library_autograd(k, s, p, hw):
    rng = np.random.default_rng(11)
    x = torch.from_numpy(rng.standard_normal((3, 4, hw, hw)))
    W = torch.from_numpy(rng.standard_normal((5, 4, k, k))).requires_grad_(True)
    y = torch.nn.functional.conv2d(x, W, stride=s, padding=p)
    delta = torch.from_numpy(rng.standard_normal(tuple(y.shape)))
    (y * delta).sum().backward()
    got = O.wgrad_plain(delta.numpy(), x.numpy(), 1.0, k, k, s, p)
    assert rel(got, W.grad.numpy()) < 1e-12


@pytest.mark.parametrize("K,kind", [(1, "fc"), (2, "fc"), (4, "conv"), (8, "conv")])
def test_wgrad_masked_equals_plain(K, kind):
    spec = tiny_fc_spec(K=K, G=3) if kind == "fc" else tiny_conv_spec(K=K, G=2, sigma=1000.0)
    d = synth.draw_layer(spec)
    xbar = O.encode(d["x"], d["r"], d["C"])
    scale = 1.0 / spec.batch
    got = O.wgrad_masked(d["delta"], xbar, d["C"], d["gamma"], scale, spec.kh, spec.kw, spec.stride, spec.pad)
    want = O.wgrad_plain(d["delta"], d["x"], scale, spec.kh, spec.kw, spec.stride, spec.pad)
    assert rel(got, want) < 1e-9
    # K+1 stored encodings per group (redundant row dropped) give the same result
    E = K + 2
    keep = np.array([g * E + j for g in range(spec.G) for j in range(K + 1)])
    got2 = O.wgrad_masked(d["delta"], xbar[keep], d["C"], d["gamma"], scale, spec.kh, spec.kw,
                          spec.stride, spec.pad, xbar_rows_per_group=K + 1)
    assert rel(got2, want) < 1e-9


def test_wgrad_fc_is_sum_of_outer_products():
    spec = tiny_fc_spec(K=2, G=2)
    d = synth.draw_layer(spec)
    want = sum(np.outer(d["delta"][b].astype(np.float64), d["x"][b].astype(np.float64)) for b in range(4))
    assert rel(O.wgrad_plain(d["delta"], d["x"], 1.0), want) < 1e-14


def test_pins_catch_gamma_applied_twice():
    spec = tiny_fc_spec(K=2, G=1)
    d = synth.draw_layer(spec)
    xbar = O.encode(d["x"], d["r"], d["C"])
    g2 = d["gamma"] * d["gamma"]
    # B derived for gamma but decoded with gamma^2: Eq. 6 no longer holds
    B = O.derive_B(d["C"][0], d["gamma"][0])
    tot = 0.0
    for j in range(3):
        dbar = sum(B[j, i] * d["delta"][i].astype(np.float64) for i in range(2))
        tot = tot + g2[0, j] * np.outer(dbar, xbar[j])
    assert rel(tot, O.wgrad_plain(d["delta"], d["x"], 1.0)) > 1e-2


# ---------------------------------------------------------------------------
# what the paper states in numbers
# ---------------------------------------------------------------------------
def test_cost_accounting_matches_paper_ratios():
    rows = [tuple(map(int, ln.split())) for ln in open(os.path.join(GOLD, "cost_ratios.txt"))
            if not ln.startswith("#")]
    for K, e_priv, e_int in rows:
        spec = tiny_conv_spec(K=K, G=3)
        plain = 2.0 * spec.cout * spec.kc * spec.batch * spec.hout * spec.wout
        assert spec.wgrad_flops() / plain == pytest.approx(e_priv / K)       # 1/K extra
        assert spec.fwd_flops() / plain == pytest.approx(e_int / K)          # one more equation
        d = synth.draw_layer(spec)
        assert O.encode(d["x"], d["r"], d["C"]).shape[0] == spec.G * e_int


def test_field_prime_is_largest_25_bit_prime():
    vals = dict(ln.split() for ln in open(os.path.join(GOLD, "field_constants.txt")) if not ln.startswith("#"))
    p = int(vals["p"])
    assert p == 2 ** 25 - 39

    def is_prime(n):
        return n > 1 and all(n % q for q in range(2, int(n ** 0.5) + 1))
    assert is_prime(p)
    assert not any(is_prime(q) for q in range(p + 1, 2 ** 25))


# ---------------------------------------------------------------------------
# input generators
# ---------------------------------------------------------------------------
def test_synth_is_seeded_and_shaped():
    spec = synth.layer("vgg16_cifar", "conv5_1").with_groups(2)
    a, b = synth.draw_layer(spec), synth.draw_layer(spec)
    for k in a:
        assert np.array_equal(a[k], b[k]) and a[k].dtype == np.float32
    assert a["x"].shape == (8, 512, 2, 2) and a["r"].shape == (2, 512, 2, 2)
    assert a["C"].shape == (2, 6, 5) and a["gamma"].shape == (2, 5)
    assert 50 < a["r"].std() < 150 and 0 <= a["x"].min() and a["x"].max() <= 1
    for wl in synth.WORKLOADS:
        for s in synth.layers(wl):
            assert s.batch == {"fc784": 2, "vgg16_cifar": 128, "resnet18_224": 64,
                               "mobilenetv2_pw": 128, "vgg16_224": 256}[wl]
    assert sum(s.fwd_flops() for s in synth.layers("vgg16_cifar")) == pytest.approx(120.3e9, rel=0.01)
    assert sum(s.fwd_flops() for s in synth.layers("vgg16_224")) == pytest.approx(11.88e12, rel=0.01)


def test_layout_permutations_roundtrip():
    rng = np.random.default_rng(12)
    a = rng.standard_normal((2, 3, 4, 5)).astype(np.float32)
    assert np.array_equal(synth.from_channels_last(synth.to_channels_last(a)), a)
    assert synth.to_channels_last(a)[1, 2, 3, 0] == a[1, 0, 2, 3]
    W = rng.standard_normal((6, 3, 3, 3)).astype(np.float32)
    assert np.array_equal(synth.weights_from_ohwi(synth.weights_to_ohwi(W)), W)
