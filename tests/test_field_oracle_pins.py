"""Pins of the finite-field oracle (Section 5 of the paper, Algorithm 1) to
things other than itself: a sieve, hand-derived values, Python's unbounded
integers, Fermat's little theorem, the unmasked product, the error bound of
the quantisation, and the one-time-pad bijection of the privacy lemma."""
import itertools
import os

import numpy as np
import pytest

from oracle import dk_field_oracle as F
from paper_2207_00083_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
P = F.P_PAPER
L = F.L_PAPER


def _spec(kind="conv", **kw):
    base = dict(workload="field_test", name="t", kind=kind, cin=5, cout=4, h=6, w=5, kh=3, kw=3, stride=1,
                pad=1, K=2, G=2)
    if kind == "fc":
        base.update(h=1, w=1, kh=1, kw=1, pad=0)
    base.update(kw)
    return synth.LayerSpec(**base)


# ---------------------------------------------------------------------------
# constants, Round, Field
# ---------------------------------------------------------------------------
def test_constants_match_the_paper_and_a_sieve():
    vals = dict(ln.split() for ln in open(os.path.join(GOLD, "field_constants.txt")) if not ln.startswith("#"))
    assert F.P_PAPER == int(vals["p"]) and F.L_PAPER == int(vals["l"])
    # sieve of Eratosthenes below 2^25: an independent route to "the largest 25-bit prime"
    n = 1 << 25
    sieve = np.ones(n, dtype=bool)
    sieve[:2] = False
    for d in range(2, int(n ** 0.5) + 1):
        if sieve[d]:
            sieve[d * d::d] = False
    assert int(np.flatnonzero(sieve)[-1]) == F.P_PAPER
    assert F.is_prime(F.P_PAPER)
    for m in (1, 4, 91, 2 ** 25 - 37, 5779 * 5783):
        assert F.is_prime(m) == bool(m < n and sieve[m]) if m < n else not F.is_prime(m)


def test_round_follows_algorithm_1_on_hand_values():
    v = np.array([0.0, 0.49, 0.5, 1.5, 2.5, -0.5, -0.51, -1.5, -2.49, 7.999])
    # fractional part below one half -> floor, otherwise floor + 1
    want = np.array([0, 0, 1, 2, 3, 0, -1, -1, -2, 8])
    assert np.array_equal(F.round_half_up(v), want)


def test_field_maps_every_integer_to_its_residue():
    v = np.array([0, 1, P - 1, P, P + 1, -1, -P, -P - 1, 3 * P + 5, -3 * P - 5, 2 ** 40, -2 ** 40])
    want = np.array([int(t) % P for t in v])      # Python's % is the mathematical residue
    got = F.to_field(v, P)
    assert np.array_equal(got, want) and got.min() >= 0 and got.max() < P


def test_quantise_centre_roundtrip_is_within_half_a_step():
    rng = np.random.default_rng(1)
    v = rng.uniform(-100, 100, 5000)
    q = F.quantize(v, L, P)
    back = F.centre(q, P).astype(np.float64) / 2 ** L
    assert np.max(np.abs(back - v)) <= 0.5 / 2 ** L + 1e-12
    # negative numbers live in the upper half of the field
    assert np.all((q > P // 2) == (F.round_half_up(v * 2 ** L) < 0))


def test_dequantize_output_on_hand_values():
    # Y_q carries 2l fractional bits; l = 2: 2^-l = 0.25
    yq = np.array([0, 1, 2, 3, 6, -2, -3, 40])
    # yq/4 = 0, .25, .5, .75, 1.5, -.5, -.75, 10 -> Round -> 0,0,1,1,2,0,-1,10 -> * 0.25
    assert np.array_equal(F.dequantize_output(yq, 2), np.array([0, 0, .25, .25, .5, 0, -.25, 2.5]))


# ---------------------------------------------------------------------------
# linear algebra in F_p
# ---------------------------------------------------------------------------
def test_inverse_agrees_with_fermat():
    rng = np.random.default_rng(2)
    for a in [1, 2, P - 1, P - 2] + list(rng.integers(1, P, 50)):
        inv = F.inv_mod(int(a), P)
        assert inv == pow(int(a), P - 2, P) and (inv * int(a)) % P == 1
    with pytest.raises(ZeroDivisionError):
        F.inv_mod(P, P)


@pytest.mark.parametrize("n", [2, 3, 5, 9])
def test_matrix_inverse_and_null_vector(n):
    rng = np.random.default_rng(n)
    M = rng.integers(0, P, (n + 1, n))
    inv = F.invert_mod(M[:n], P)
    prod = [[sum(int(M[i, k]) * int(inv[k, j]) for k in range(n)) % P for j in range(n)] for i in range(n)]
    assert prod == [[int(i == j) for j in range(n)] for i in range(n)]
    nv = F.null_vector_mod(M, P)
    assert nv[n] == 1
    assert all(sum(int(nv[i]) * int(M[i, k]) for i in range(n + 1)) % P == 0 for k in range(n))
    sing = M[:n].copy()
    sing[1] = (3 * sing[0]) % P
    with pytest.raises(np.linalg.LinAlgError):
        F.invert_mod(sing, P)


# ---------------------------------------------------------------------------
# contractions against Python-integer brute force
# ---------------------------------------------------------------------------
def _brute_conv(Wq, xq, p, stride, pad):
    n, cin, h, w = xq.shape
    cout, _, kh, kw = Wq.shape
    ho, wo = (h + 2 * pad - kh) // stride + 1, (w + 2 * pad - kw) // stride + 1
    out = np.zeros((n, cout, ho, wo), dtype=np.int64)
    for s, o, a, b in itertools.product(range(n), range(cout), range(ho), range(wo)):
        acc = 0
        for c, u, v in itertools.product(range(cin), range(kh), range(kw)):
            ih, iw = a * stride + u - pad, b * stride + v - pad
            if 0 <= ih < h and 0 <= iw < w:
                acc += int(Wq[o, c, u, v]) * int(xq[s, c, ih, iw])
        out[s, o, a, b] = acc % p
    return out


@pytest.mark.parametrize("stride,pad", [(1, 1), (2, 0), (2, 1)])
def test_field_linear_conv_against_brute_force(stride, pad):
    rng = np.random.default_rng(10 + stride + pad)
    Wq = rng.integers(0, P, (3, 4, 3, 3))
    xq = rng.integers(0, P, (2, 4, 6, 5))
    assert np.array_equal(F.field_linear(Wq, xq, P, stride, pad), _brute_conv(Wq, xq, P, stride, pad))


def test_field_linear_fc_long_contraction_against_python_integers():
    # longer than one int64-safe piece (2^63 / p^2 is about 8191 terms)
    rng = np.random.default_rng(3)
    kc = 20000
    Wq = rng.integers(P - 1000, P, (2, kc))      # near-maximal residues: the worst case for overflow
    xq = rng.integers(P - 1000, P, (3, kc))
    got = F.field_linear(Wq, xq, P)
    want = [[sum(int(a) * int(b) for a, b in zip(xq[s], Wq[o])) % P for o in range(2)] for s in range(3)]
    assert got.tolist() == want


def test_field_wgrad_against_brute_force():
    rng = np.random.default_rng(4)
    cout, cin, h, w, kh, kw, stride, pad = 3, 2, 5, 6, 3, 3, 2, 1
    ho, wo = (h + 2 * pad - kh) // stride + 1, (w + 2 * pad - kw) // stride + 1
    d = rng.integers(0, P, (cout, ho, wo))
    x = rng.integers(0, P, (cin, h, w))
    got = F.field_bilinear_wgrad(d, x, P, kh, kw, stride, pad)
    for o, c, u, v in itertools.product(range(cout), range(cin), range(kh), range(kw)):
        acc = 0
        for a, b in itertools.product(range(ho), range(wo)):
            ih, iw = a * stride + u - pad, b * stride + v - pad
            if 0 <= ih < h and 0 <= iw < w:
                acc += int(d[o, a, b]) * int(x[c, ih, iw])
        assert got[o, c, u, v] == acc % P
    # FC: outer product
    dv, xv = rng.integers(0, P, 4), rng.integers(0, P, 5)
    assert F.field_bilinear_wgrad(dv, xv, P).tolist() == [[int(a) * int(b) % P for b in xv] for a in dv]


# ---------------------------------------------------------------------------
# the method's invariants
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("kind,K", [("fc", 1), ("fc", 4), ("conv", 2), ("conv", 3)])
def test_decode_of_linear_of_encode_is_the_plain_product(kind, K):
    spec = _spec(kind, K=K, G=2)
    d = synth.draw_field_layer(spec, P)
    Wq, xq = F.quantize(d["W"], L, P), F.quantize(d["x"], L, P)
    xbar = F.field_encode(xq, d["rq"], d["Cq"], P)
    ybar = F.field_linear(Wq, xbar, P, spec.stride, spec.pad)
    yq, zq = F.field_decode(ybar, d["Cq"], P)
    assert np.array_equal(yq, F.field_linear_plain(Wq, xq, P, spec.stride, spec.pad))
    assert np.array_equal(zq, F.field_linear_plain(Wq, d["rq"], P, spec.stride, spec.pad))
    assert not F.field_verify(ybar, d["Cq"], yq, zq, P).any()
    # taking the centred representatives of y_bar before decoding changes nothing modulo p
    y2, _ = F.field_decode(F.to_field(F.centre(ybar, P), P), d["Cq"], P)
    assert np.array_equal(y2, yq)


def test_encoding_brute_force_and_transposed_coefficients_differ():
    spec = _spec("fc", K=2, G=1, cin=3)
    d = synth.draw_field_layer(spec, P)
    xq = F.quantize(d["x"], L, P)
    got = F.field_encode(xq, d["rq"], d["Cq"], P)
    C = d["Cq"][0]
    for i in range(4):
        for e in range(3):
            want = (int(C[i, 0]) * int(xq[0, e]) + int(C[i, 1]) * int(xq[1, e]) + int(C[i, 2]) * int(d["rq"][0, e])) % P
            assert got[i, e] == want


def test_single_fault_is_flagged_exactly_where_it_was_injected():
    spec = _spec("conv", K=3, G=2)
    d = synth.draw_field_layer(spec, P)
    clean = F.field_masked_forward(d["W"], d["x"], d["rq"], d["Cq"], L, P, spec.stride, spec.pad)
    assert not clean["flags"].any()
    for enc in range(spec.K + 2):
        e = 17 + enc
        bad = F.field_masked_forward(d["W"], d["x"], d["rq"], d["Cq"], L, P, spec.stride, spec.pad,
                                     fault=(1, enc, e, 1))
        v = F.field_verdict(bad["flags"])
        assert v == {"ok": 0, "n_flagged": 1, "first_index": spec.n_out + e}
        # the residual of the redundant equation moves by n[enc] * fault (no zero divisors in F_p)
        n = F.null_vector_mod(d["Cq"][1], P)
        E = spec.K + 2
        rho = sum(int(n[i]) * int(bad["ybar"][E + i].reshape(-1)[e]) for i in range(E)) % P
        assert rho == int(n[enc]) % P and rho != 0


def test_whole_procedure_is_within_the_quantisation_bound_of_the_float_product():
    spec = _spec("conv", K=2, G=2, cin=8, cout=6)
    d = synth.draw_field_layer(spec, P)
    out = F.field_masked_forward(d["W"], d["x"], d["rq"], d["Cq"], L, P, spec.stride, spec.pad, bias=d["bias"])
    W, x = d["W"].astype(np.float64), d["x"].astype(np.float64)
    # plain float64 cross-correlation by a library routine
    import torch
    want = torch.nn.functional.conv2d(torch.from_numpy(x), torch.from_numpy(W), torch.from_numpy(d["bias"].astype(np.float64)),
                                      stride=spec.stride, padding=spec.pad).numpy()
    h = 0.5 / 2 ** L          # rounding error of one quantised value
    bound = spec.kc * (np.abs(W).max() * h + np.abs(x).max() * h + h * h) + h * h + h
    err = np.max(np.abs(out["y"] - want))
    assert err <= bound and err > 0
    # and no wrap-around happened: the integers stayed inside (-p/2, p/2)
    assert np.abs(want).max() * 4 ** L < P / 2


def test_decoded_integers_equal_the_integer_product_when_it_fits():
    # small integers: the centred decoded value is the true (not reduced) integer product
    rng = np.random.default_rng(6)
    K, G = 2, 1
    Wi = rng.integers(-50, 50, (3, 7))
    xi = rng.integers(-50, 50, (G * K, 7))
    Cq = rng.integers(1, P, (G, K + 2, K + 1))
    rq = rng.integers(0, P, (G, 7))
    ybar = F.field_linear(F.to_field(Wi, P), F.field_encode(F.to_field(xi, P), rq, Cq, P), P)
    yq, _ = F.field_decode(ybar, Cq, P)
    assert np.array_equal(F.centre(yq, P), xi @ Wi.T)


def test_eq5_holds_in_the_field_and_masked_wgrad_is_the_plain_one():
    for kind in ("fc", "conv"):
        spec = _spec(kind, K=3, G=2, stride=2 if kind == "conv" else 1)
        d = synth.draw_field_layer(spec, P)
        K1 = spec.K + 1
        for g in range(spec.G):
            B = F.field_derive_B(d["Cq"][g], d["gammaq"][g], P)
            A = d["Cq"][g][:K1].T                      # the paper's A (sources x encodings)
            # B^T . Gamma . A^T = [I_K | 0]
            for i in range(spec.K):
                for k in range(K1):
                    s = sum(int(B[j, i]) * int(d["gammaq"][g, j]) * int(A[k, j]) for j in range(K1)) % P
                    assert s == int(i == k)
        xq, dq = F.quantize(d["x"], L, P), F.quantize(d["delta"], L, P)
        xbar = F.field_encode(xq, d["rq"], d["Cq"], P)
        got = F.field_wgrad_masked(dq, xbar, d["Cq"], d["gammaq"], P, spec.kh, spec.kw, spec.stride, spec.pad)
        want = F.field_wgrad_plain(dq, xq, P, spec.kh, spec.kw, spec.stride, spec.pad)
        assert np.array_equal(got, want)
        # a wrong gamma breaks it (the coefficient must be used on both sides)
        g2 = d["gammaq"].copy()
        B_wrong = F.field_derive_B(d["Cq"][0], g2[0], P)
        g2[0, 0] = (g2[0, 0] + 1) % P
        term = F.field_wgrad_masked(dq, xbar, d["Cq"], d["gammaq"], P, spec.kh, spec.kw, spec.stride, spec.pad,
                                    xbar_rows=spec.K + 2)
        assert np.array_equal(term, want) and B_wrong.shape == (K1, spec.K)


def test_one_time_pad_bijection_on_a_tiny_field():
    # Lemma 1: x + z with z uniform over F_p is uniform.  On F_11 with any non-zero
    # noise coefficient the encoded value runs through the whole field exactly once as r does.
    p = 11
    for c_noise in range(1, p):
        Cq = np.array([[[3, c_noise], [5, 1], [2, 7]]])
        seen = sorted(int(F.field_encode(np.array([[4]]), np.array([[r]]), Cq, p)[0, 0]) for r in range(p))
        assert seen == list(range(p))


def test_single_element_functions_agree_with_the_full_ones():
    spec = _spec("conv", K=2, G=2, stride=2, pad=1)
    d = synth.draw_field_layer(spec, P)
    Wq, xq, dq = F.quantize(d["W"], L, P), F.quantize(d["x"], L, P), F.quantize(d["delta"], L, P)
    full = F.field_linear(Wq, xq, P, spec.stride, spec.pad)
    fullw = F.field_wgrad_plain(dq, xq, P, spec.kh, spec.kw, spec.stride, spec.pad)
    for s, co, oh, ow in [(0, 0, 0, 0), (3, 3, spec.hout - 1, spec.wout - 1), (2, 1, 1, 2)]:
        assert F.field_linear_at(Wq, xq[s], co, oh, ow, P, spec.stride, spec.pad) == full[s, co, oh, ow]
    for co, ci, u, v in [(0, 0, 0, 0), (3, 4, 2, 2), (1, 2, 0, 1)]:
        assert F.field_wgrad_plain_at(dq, xq, co, ci, u, v, P, spec.stride, spec.pad) == fullw[co, ci, u, v]
    fc = _spec("fc", K=2, G=2)
    d = synth.draw_field_layer(fc, P)
    Wq, xq, dq = F.quantize(d["W"], L, P), F.quantize(d["x"], L, P), F.quantize(d["delta"], L, P)
    assert F.field_linear_at(Wq, xq[1], 2, 0, 0, P) == F.field_linear(Wq, xq, P)[1, 2]
    assert F.field_wgrad_plain_at(dq, xq, 3, 1, 0, 0, P) == F.field_wgrad_plain(dq, xq, P)[3, 1]
