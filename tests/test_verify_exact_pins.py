"""Pins of the integrity rules to the one thing Section 4.4 fixes: results that
are "not consistent" are flagged, which in exact arithmetic means residual != 0.

The floating-point oracle compares |rho| with tau * max(s_e, s_g); the paper
compares exactly in F_p.  On inputs made of small integers with a unimodular
square coefficient block (integer inverse) the true residual is an integer and
the oracle's fp64 residual is off by ~1e-13 at most (its Gauss-Jordan inverse
divides by pivots), ten orders of magnitude below tau * scale; so its flag set
must be exactly {e : rho_e != 0}, where rho is computed here independently in
integers, and it must equal the flag set of the finite-field oracle for the
same integers taken modulo p.  A dropped
term, a wrong sign or a wrong index in the residual, the null vector or either
normaliser makes an honest element non-zero or a faulted one zero and fails.

The same is done for the weight-gradient check (two equation sets, Eq. 4-6):
with gamma = +-1 the true gradients are integers, so an element is flagged iff
the two decoded gradients differ (closed form of the difference computed here).
"""
import numpy as np
import pytest

from oracle import dk_field_oracle as F
from oracle import dk_oracle as O

P = F.P_PAPER
TAU = 1e-4


def unimodular(rng, n):
    """Integer matrix with determinant +-1: a product of elementary row operations."""
    M = np.eye(n, dtype=np.int64)
    for _ in range(3 * n):
        i, j = rng.choice(n, 2, replace=False) if n > 1 else (0, 0)
        if i != j:
            M[i] += int(rng.integers(-2, 3)) * M[j]
    if rng.integers(0, 2) and n > 1:
        M[[0, 1]] = M[[1, 0]]
    return M


def integer_case(seed, K, G, kind):
    """Small-integer layer: C with unimodular square part and a redundant row whose null vector has no
    zero component, x, r, W integers."""
    rng = np.random.default_rng(seed)
    C = np.zeros((G, K + 2, K + 1), dtype=np.int64)
    for g in range(G):
        while True:
            sq = unimodular(rng, K + 1)
            red = rng.integers(-3, 4, K + 1)
            # null vector over the integers: n[:K+1] = -red . sq^{-1} (integer because det = +-1)
            inv = np.rint(np.linalg.inv(sq.astype(np.float64))).astype(np.int64)
            assert np.array_equal(sq @ inv, np.eye(K + 1, dtype=np.int64))
            n = -(red @ inv)
            if np.all(n != 0) and np.all(sq[:, K] != 0) and np.max(np.abs(sq)) <= 12:
                C[g, :K + 1], C[g, K + 1] = sq, red
                break
    if kind == "fc":
        cin, cout = 6, 5
        x = rng.integers(-2, 3, (G * K, cin))
        r = rng.integers(-4, 5, (G, cin))
        W = rng.integers(-1, 2, (cout, cin))
        geo = dict(stride=1, pad=0)
    else:
        cin, cout = 3, 4
        x = rng.integers(-2, 3, (G * K, cin, 5, 4))
        r = rng.integers(-4, 5, (G, cin, 5, 4))
        W = rng.integers(-1, 2, (cout, cin, 3, 3))
        geo = dict(stride=1, pad=1)
    return C, x, r, W, geo


def exact_null_vector(Cg):
    K1 = Cg.shape[1]
    inv = np.rint(np.linalg.inv(Cg[:K1].astype(np.float64))).astype(np.int64)
    return np.concatenate([-(Cg[K1] @ inv), [1]])


def exact_residual(ybar_int, C):
    """rho[g] = sum_i n_g[i] * ybar[g*E + i] in Python-exact int64 (values are tiny)."""
    G, E, _ = C.shape
    return np.stack([sum(int(n) * ybar_int[g * E + i] for i, n in enumerate(exact_null_vector(C[g])))
                     for g in range(G)])


CASES = [(1, 1, 2, "fc"), (2, 2, 2, "fc"), (3, 4, 1, "fc"), (4, 2, 2, "conv"), (5, 3, 1, "conv"), (6, 8, 1, "fc")]


@pytest.mark.parametrize("seed,K,G,kind", CASES)
def test_float_rule_flags_exactly_the_nonzero_residuals_and_agrees_with_the_field_rule(seed, K, G, kind):
    C, x, r, W, geo = integer_case(seed, K, G, kind)
    E = K + 2
    xbar = O.encode(x, r, C)
    ybar = O.linear(W, xbar, **geo)
    assert np.array_equal(ybar, np.rint(ybar))                 # exact so far
    ybar_int = ybar.astype(np.int64)
    assert not exact_residual(ybar_int, C).any()               # honest run: rho == 0 (the paper's identity)

    rng = np.random.default_rng(100 + seed)
    n_el = ybar[0].size
    shape = ybar.shape[1:]
    # faults: elements in different encodings (two may share an element without cancelling), and a
    # crafted pair on one element that cancels in the redundant equation (undetectable by ANY consistency
    # check of these K+2 equations, in the paper's exact rule as well)
    faults = []
    for g in range(G):
        for i in rng.choice(E, size=min(E, 3), replace=False):
            e = int(rng.integers(0, n_el))
            faults.append((g, int(i), e, int(rng.choice([-3, -1, 1, 2, 5]))))
    g0 = 0
    n0 = exact_null_vector(C[g0])
    e_cancel = next(e for e in range(n_el) if all(f[2] != e for f in faults if f[0] == g0))
    faults.append((g0, 0, e_cancel, int(n0[1])))
    faults.append((g0, 1, e_cancel, -int(n0[0])))              # n0[0]*n0[1] - n0[1]*n0[0] == 0
    bad = ybar.copy()
    for g, i, e, dlt in faults:
        bad[g * E + i][np.unravel_index(e, shape)] += dlt
    bad_int = bad.astype(np.int64)

    rho = exact_residual(bad_int, C)
    want = rho != 0
    assert not want[g0][np.unravel_index(e_cancel, shape)]     # the cancelling pair leaves rho == 0
    assert want.sum() >= G                                     # and the other faults do not

    y, z = O.decode(bad, C)
    chk = O.verify(bad, C, y, z, tau=TAU)
    # precondition under which "nonzero" and "above threshold" coincide: |rho| >= 1 > tau * scale
    assert float(chk["scale"].max()) < 1.0 / TAU
    # the oracle's residual is the exact one up to the rounding of its Gauss-Jordan inverse, ten orders
    # of magnitude below the threshold: the decision is the exact rule's
    assert np.max(np.abs(chk["rho"] - rho)) < 1e-9
    assert np.array_equal(chk["flags"], want)

    # the paper's own rule, on the same integers modulo p
    badq = np.mod(bad_int, P)
    Cq = np.mod(C, P)
    yq, zq = F.field_decode(badq, Cq, P)
    assert np.array_equal(F.field_verify(badq, Cq, yq, zq, P), want)
    # the decoded values are the same integers on both sides (an integer inverse keeps fp64 exact)
    assert np.max(np.abs(y - np.rint(y))) < 1e-9
    assert np.array_equal(F.centre(yq, P), np.rint(y).astype(np.int64))


@pytest.mark.parametrize("seed,K,G,kind", CASES[:5])
def test_group_term_never_hides_an_exact_inconsistency(seed, K, G, kind):
    """max(s_e, s_g) instead of s_e alone raises the floor at elements whose encodings are all small;
    with exact arithmetic and |rho| >= 1 the decision must still be 'flagged' while s_g < 1/tau, and
    an element whose every encoded output is zero (s_e == 0) is decided by s_g alone."""
    C, x, r, W, geo = integer_case(seed, K, G, kind)
    E = K + 2
    W = W.copy()
    W[0] = 0                                                   # output channel 0: every y_bar is zero there
    ybar = O.linear(W, O.encode(x, r, C), **geo)
    idx = (0,) if kind == "fc" else (0, 1, 1)
    assert all(ybar[i][idx] == 0 for i in range(G * E))
    bad = ybar.copy()
    bad[1][idx] += 1.0                                         # encoding 1 of group 0
    y, z = O.decode(bad, C)
    chk = O.verify(bad, C, y, z, tau=TAU)
    n = exact_null_vector(C[0])
    assert abs(chk["rho"][0][idx] - float(n[1])) < 1e-9
    assert chk["scale"][0][idx] >= abs(n[1]) - 1e-9            # s_e = |n_1| * 1, s_g may exceed it
    assert chk["flags"].sum() == 1 and chk["flags"][0][idx]


WG_CASES = [(11, 2, 2, "fc"), (12, 3, 1, "fc"), (13, 2, 1, "conv"), (14, 1, 2, "conv")]


@pytest.mark.parametrize("seed,K,G,kind", WG_CASES)
def test_wgrad_check_flags_exactly_where_the_two_equation_sets_differ(seed, K, G, kind):
    C, x, r, W, geo = integer_case(seed, K, G, kind)
    rng = np.random.default_rng(200 + seed)
    gamma = rng.choice([-1.0, 1.0], size=(G, K + 1))
    xbar = O.encode(x, r, C)
    cout = W.shape[0]
    if kind == "fc":
        delta = rng.integers(-2, 3, (G * K, cout)).astype(np.float64)
        kh = kw = 1
    else:
        delta = rng.integers(-2, 3, (G * K, cout, 5, 4)).astype(np.float64)
        kh = kw = 3
    st, pad = geo["stride"], geo["pad"]
    clean = O.wgrad_redundant(delta, xbar, C, gamma, 1.0, kh, kw, st, pad, tau_w=1e-2)
    plain = O.wgrad_plain(delta, x, 1.0, kh, kw, st, pad)
    assert np.array_equal(plain, np.rint(plain))
    assert np.max(np.abs(clean["dW"] - plain)) < 1e-8 and np.max(np.abs(clean["dW_second"] - plain)) < 1e-8
    assert not clean["flags"].any()
    assert 1e-2 * clean["rms"] < 0.5                           # an integer difference is above the threshold
    # One wrong encoded activation, used by the first set only (encoding 0 of group 0).  The first
    # result moves by gamma_0 <delta_bar_0, 3 e_pos> = 3 <sum_i inv[i][0] delta_i, e_pos> with the INTEGER
    # inverse of the square block (computed here, not by the oracle); the second set does not see it.
    xb = xbar.copy()
    pos = (2,) if kind == "fc" else (1, 2, 2)
    xb[0][pos] += 3.0
    inv = np.rint(np.linalg.inv(C[0, :K + 1].astype(np.float64))).astype(np.int64)
    mixed = sum(int(inv[i, 0]) * delta[i].astype(np.int64) for i in range(K))      # delta_bar_0 * gamma_0
    diff = np.zeros(plain.shape, dtype=np.int64)
    if kind == "fc":
        diff[:, pos[0]] = 3 * mixed
    else:
        c0, y0, x0 = pos
        for u in range(kh):
            for v in range(kw):
                p_, q_ = y0 - u + pad, x0 - v + pad
                if 0 <= p_ < mixed.shape[1] and 0 <= q_ < mixed.shape[2]:
                    diff[:, c0, u, v] = 3 * mixed[:, p_, q_]
    want = diff != 0
    assert want.any()
    bad = O.wgrad_redundant(delta, xb, C, gamma, 1.0, kh, kw, st, pad, tau_w=1e-2)
    assert np.max(np.abs(bad["dW_second"] - plain)) < 1e-8
    assert np.max(np.abs(bad["dW"] - plain - diff)) < 1e-8
    assert np.array_equal(bad["flags"], want)
