"""fp64 CPU oracle for DarKnight's masked linear-algebra path.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
path computes, written from the paper; it shares no code with the CUDA
library and must never be imported by it.  Only the tests, the smoke check
and the benchmark's CPU-baseline leg call it.

Every function works on float64 NumPy arrays in the paper's logical shapes
(samples first, then channels, then rows, columns) and follows the paper's
steps in order, without blocking or fusion:

* ``encode``            Eq. 1, plus the redundant encoding of Section 4.4
* ``linear``            the bilinear operation <W, x> (matrix product or
                        cross-correlation with zero padding), Section 4.1
* ``decode``            Eq. 2: Y = Y_bar . A^{-1}; the W.r column is returned
                        separately and dropped by the caller
* ``verify``            Section 4.4: the (K+2)-th equation is re-predicted from
                        the decoded unknowns and compared with what came back
* ``derive_B``          the unique B that satisfies Eq. 5 for given A, Gamma
* ``wgrad_masked``      Eq. 4 and Eq. 6, summed over virtual batches
* ``linear_plain`` / ``wgrad_plain``   the unmasked definitions (Eq. 3) that
                        the method must reproduce exactly in exact arithmetic
* ``wgrad_redundant``   the "two sets of equations" idea of Section 4.4 applied
                        to the weight gradient: decode it from encodings
                        1..K+1 and again from encodings 2..K+2, compare
* ``dgrad_plain`` / ``relu`` / ``relu_bwd`` / ``maxpool2x2`` / ``maxpool2x2_bwd`` /
  ``training_step_plain``   the unmasked steps that chain the masked products
                        into a training step (Section 4.2 back-propagation of
                        delta "without encoding", the non-linear layers of the
                        Section 3.1 flow, Section 6 aggregation)
* ``encode_colluding`` / ``decode_colluding`` / ``wgrad_colluding`` /
  ``colluding_subsets_full_rank``   the M-noise-vector scheme of Section 4.5
                        (X_bar = X.A1 + R.A2, S = K + M encodings)

Coefficient convention: ``C[g, i, k]`` = coefficient of source k (k < K the
private inputs, k = K the noise) in encoding i; rows 0..K are the decodable
square part C_sq (the transpose of the paper's A), row K+1 is the redundant
row.

Pins (see the ``-m "not gpu"`` tests): brute-force loops on tiny inputs, a
library float64 convolution and its autograd, the decode/encode round trip
against the plain definition, closed forms for K = 1, the exact residual
change n[i]*Delta under a single injected fault, the Eq. 5 residual, the exact
(integer) residuals and the finite-field flag set on small-integer inputs for
both integrity rules, and float64 autograd of a library three-layer chain for
the back-propagation helpers.
Parity unpinned: the numerical VALUE of the threshold ``tau`` of ``verify`` and
of ``tau_w`` of ``wgrad_redundant`` (a check the paper does not describe for the
backward pass) and the choice of normalisers max(s_e, s_g) and rms(dW) are
choices of this implementation, not the paper's (the paper compares exactly in
a finite field).  What the paper does fix is pinned: with exact arithmetic
both rules flag exactly the elements whose residual is non-zero, and the
first agrees with the finite-field rule on the same integers.
"""
from __future__ import annotations

from typing import Dict, Optional, Tuple

import numpy as np

F64 = np.float64


# ---------------------------------------------------------------------------
# small dense linear algebra, written out (no library inverse)
# ---------------------------------------------------------------------------
def invert(M: np.ndarray) -> np.ndarray:
    """Gauss-Jordan inverse with partial pivoting of a small square matrix."""
    n = M.shape[0]
    a = np.array(M, dtype=F64)
    inv = np.eye(n, dtype=F64)
    for col in range(n):
        piv = col + int(np.argmax(np.abs(a[col:, col])))
        if a[piv, col] == 0.0:
            raise ZeroDivisionError("singular coefficient matrix")
        if piv != col:
            a[[col, piv]] = a[[piv, col]]
            inv[[col, piv]] = inv[[piv, col]]
        p = a[col, col]
        a[col] /= p
        inv[col] /= p
        for row in range(n):
            if row != col and a[row, col] != 0.0:
                f = a[row, col]
                a[row] -= f * a[col]
                inv[row] -= f * inv[col]
    return inv


def null_vector(Cg: np.ndarray) -> np.ndarray:
    """n with n^T C = 0 and n[K+1] = 1 for a (K+2)x(K+1) block (Section 4.4).

    Any consistency check between two (K+1)-subsets of the K+2 equations is a
    multiple of n . y_bar, because the left null space of C has dimension one.
    """
    K1 = Cg.shape[1]
    c = np.asarray(Cg, dtype=F64)
    n = np.empty(K1 + 1, dtype=F64)
    n[:K1] = -(c[K1] @ invert(c[:K1]))
    n[K1] = 1.0
    return n


# ---------------------------------------------------------------------------
# Eq. 1 / Section 4.4: encoding
# ---------------------------------------------------------------------------
def encode(x: np.ndarray, r: np.ndarray, C: np.ndarray) -> np.ndarray:
    """x_bar[g*(K+2)+i] = sum_k C[g,i,k] x[g*K+k] + C[g,i,K] r[g]  (Eq. 1)."""
    G, E, K1 = C.shape
    K = K1 - 1
    x = np.asarray(x, dtype=F64)
    r = np.asarray(r, dtype=F64)
    c = np.asarray(C, dtype=F64)
    out = np.zeros((G * E,) + x.shape[1:], dtype=F64)
    for g in range(G):
        for i in range(E):
            acc = c[g, i, K] * r[g]
            for k in range(K):
                acc = acc + c[g, i, k] * x[g * K + k]
            out[g * E + i] = acc
    return out


# ---------------------------------------------------------------------------
# the bilinear operation <W, x>
# ---------------------------------------------------------------------------
def _pad(x: np.ndarray, pad: int) -> np.ndarray:
    if pad == 0:
        return x
    return np.pad(x, ((0, 0), (0, 0), (pad, pad), (pad, pad)))


def linear(W: np.ndarray, x: np.ndarray, stride: int = 1, pad: int = 0) -> np.ndarray:
    """<W, x> per sample: x @ W^T for 2-D x, else zero-padded cross-correlation
    y[n,o,p,q] = sum_{c,u,v} W[o,c,u,v] x[n,c,p*stride+u-pad,q*stride+v-pad]."""
    W = np.asarray(W, dtype=F64)
    x = np.asarray(x, dtype=F64)
    if x.ndim == 2:
        return x @ W.T
    n, cin, h, w = x.shape
    cout, _, kh, kw = W.shape
    ho = (h + 2 * pad - kh) // stride + 1
    wo = (w + 2 * pad - kw) // stride + 1
    xp = _pad(x, pad)
    y = np.zeros((n, cout, ho, wo), dtype=F64)
    for u in range(kh):
        for v in range(kw):
            win = xp[:, :, u:u + (ho - 1) * stride + 1:stride, v:v + (wo - 1) * stride + 1:stride]
            # sum over channels c: y[n,o,p,q] += W[o,c,u,v] * win[n,c,p,q]
            y += np.tensordot(win, W[:, :, u, v], axes=([1], [1])).transpose(0, 3, 1, 2)
    return y


def linear_at(W: np.ndarray, x_one: np.ndarray, co: int, oh: int, ow: int,
              stride: int = 1, pad: int = 0) -> float:
    """One output element of ``linear`` for one sample (x_one has no batch axis).
    Only the filter row and the input columns under it are converted to
    float64, so that a single element of a large layer stays cheap."""
    if x_one.ndim == 1:
        return float(np.asarray(W[co], dtype=F64) @ np.asarray(x_one, dtype=F64))
    cin, h, w = x_one.shape
    _, _, kh, kw = W.shape
    acc = 0.0
    for u in range(kh):
        ih = oh * stride + u - pad
        if ih < 0 or ih >= h:
            continue
        for v in range(kw):
            iw = ow * stride + v - pad
            if iw < 0 or iw >= w:
                continue
            acc += float(np.asarray(W[co, :, u, v], dtype=F64) @ np.asarray(x_one[:, ih, iw], dtype=F64))
    return acc


def linear_plain(W, x, stride=1, pad=0):
    """The result the method must reproduce: y^(k) = <W, x^(k)> (Section 4.1)."""
    return linear(W, x, stride, pad)


# ---------------------------------------------------------------------------
# Eq. 2: decoding
# ---------------------------------------------------------------------------
def decode(ybar: np.ndarray, C: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Solve C_sq . [y^(1..K); z] = y_bar^(1..K+1) per group and element.

    Because y_bar^(i) = sum_k C[i,k] <W,x^(k)> + C[i,K] <W,r>, stacking the
    first K+1 encodings gives Y_bar = C_sq . Y (the transpose of Eq. 2), hence
    Y = C_sq^{-1} . Y_bar.  Returns (y [G*K,...], z [G,...]) with z = <W, r>.
    """
    G, E, K1 = C.shape
    K = K1 - 1
    ybar = np.asarray(ybar, dtype=F64)
    y = np.zeros((G * K,) + ybar.shape[1:], dtype=F64)
    z = np.zeros((G,) + ybar.shape[1:], dtype=F64)
    for g in range(G):
        cinv = invert(np.asarray(C[g, :K1], dtype=F64))
        for k in range(K1):
            acc = 0.0
            for i in range(K1):
                acc = acc + cinv[k, i] * ybar[g * E + i]
            if k < K:
                y[g * K + k] = acc
            else:
                z[g] = acc
    return y, z


# ---------------------------------------------------------------------------
# Section 4.4: integrity
# ---------------------------------------------------------------------------
def verify(ybar: np.ndarray, C: np.ndarray, y: np.ndarray, z: np.ndarray,
           tau: float = 1e-4) -> Dict[str, np.ndarray]:
    """Re-predict the redundant equation from the decoded unknowns.

    rho[g] = y_bar^(K+2) - sum_k C[K+1,k] y^(k) - C[K+1,K] z, which is zero in
    exact arithmetic on an honest run.  In floating point it is compared with
    the scale of the numbers it was formed from.  With n the null vector of
    the group's C,

        s_e = sum_i |n_i| |y_bar^(i)[e]|           (this element)
        s_g = sum_i |n_i| rms_e(y_bar^(i))          (the group's whole sample)

    an element is flagged iff NOT(|rho| <= tau * max(s_e, s_g)).  The group
    term is needed because all K+2 encodings share the term <W, r>: where it
    happens to be near zero every y_bar^(i)[e] is small at once while the
    rounding error of the contraction is not.  Writing the test as NOT(<=)
    flags a NaN returned by the accelerator; an element whose s_e is not
    finite is flagged as well, and non-finite values are left out of the rms.
    The comparison itself is taken in float32 (the precision in which the GPU
    takes it).

    Returns per-element arrays of shape [G, ...]: ``rho``, ``scale`` =
    max(s_e, s_g), ``ratio`` = |rho|/scale (what is compared with tau),
    ``ratio_group`` = |rho|/s_g (what the verdict reports as max_ratio) and
    boolean ``flags``.
    """
    G, E, K1 = C.shape
    K = K1 - 1
    ybar = np.asarray(ybar, dtype=F64)
    rho = np.zeros((G,) + ybar.shape[1:], dtype=F64)
    scale = np.zeros_like(rho)
    sgroup = np.zeros_like(rho)
    for g in range(G):
        c = np.asarray(C[g], dtype=F64)
        pred = c[K + 1, K] * z[g]
        for k in range(K):
            pred = pred + c[K + 1, k] * y[g * K + k]
        rho[g] = ybar[g * E + K + 1] - pred
        n = null_vector(c)
        s_e = 0.0
        s_g = 0.0
        for i in range(E):
            row = ybar[g * E + i]
            s_e = s_e + abs(n[i]) * np.abs(row)
            fin = np.isfinite(row)
            s_g = s_g + abs(n[i]) * np.sqrt(np.mean(np.where(fin, row, 0.0) ** 2))
        sgroup[g] = s_g
        with np.errstate(invalid="ignore"):
            scale[g] = np.fmax(s_e, s_g)
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(scale > 0, np.abs(rho) / scale, 0.0)
        ratio_group = np.where(sgroup > 0, np.abs(rho) / sgroup, 0.0)
        flags = ~(np.abs(rho).astype(np.float32) <= np.float32(tau) * scale.astype(np.float32))
        flags |= ~np.isfinite(scale)
    return {"rho": rho, "scale": scale, "ratio": ratio, "ratio_group": ratio_group, "flags": flags}


def verdict(flags: np.ndarray, ratio: np.ndarray) -> Dict[str, float]:
    """Summary of a verify pass over arrays given in the memory order of the
    output tensor: ok, n_flagged, first flagged flat index (-1 if none) and
    the largest ratio (NaNs ignored)."""
    flat = np.flatnonzero(np.asarray(flags).reshape(-1))
    return {"ok": int(flat.size == 0), "n_flagged": int(flat.size),
            "first_index": int(flat[0]) if flat.size else -1,
            "max_ratio": float(np.nanmax(ratio)) if ratio.size else 0.0}


# ---------------------------------------------------------------------------
# Eq. 4-6: weight gradient on encoded activations
# ---------------------------------------------------------------------------
def derive_B(Cg: np.ndarray, gamma_g: np.ndarray) -> np.ndarray:
    """B in R^{(K+1) x K} with B^T . Gamma . A^T = [I_K | 0]  (Eq. 5).

    With A square and invertible the solution is unique:
    B = Gamma^{-1} . A^{-1} . [I_K; 0].  Since C_sq = A^T this reads
    B[j,i] = (C_sq^{-1})[i,j] / gamma[j].
    """
    K1 = Cg.shape[1]
    K = K1 - 1
    cinv = invert(np.asarray(Cg[:K1], dtype=F64))
    B = np.zeros((K1, K), dtype=F64)
    for j in range(K1):
        for i in range(K):
            B[j, i] = cinv[i, j] / float(gamma_g[j])
    return B


def bilinear_wgrad(delta_one: np.ndarray, x_one: np.ndarray, kh: int = 1, kw: int = 1,
                   stride: int = 1, pad: int = 0) -> np.ndarray:
    """<delta, x> for one sample: the outer product for vectors, else
    dW[o,c,u,v] = sum_{p,q} delta[o,p,q] x[c,p*stride+u-pad,q*stride+v-pad]."""
    d = np.asarray(delta_one, dtype=F64)
    x = np.asarray(x_one, dtype=F64)
    if x.ndim == 1:
        return np.outer(d, x)
    cout, ho, wo = d.shape
    cin = x.shape[0]
    xp = _pad(x[None], pad)[0]
    dW = np.zeros((cout, cin, kh, kw), dtype=F64)
    for u in range(kh):
        for v in range(kw):
            win = xp[:, u:u + (ho - 1) * stride + 1:stride, v:v + (wo - 1) * stride + 1:stride]
            dW[:, :, u, v] = np.tensordot(d, win, axes=([1, 2], [1, 2]))
    return dW


def wgrad_masked(delta: np.ndarray, xbar: np.ndarray, C: np.ndarray, gamma: np.ndarray,
                 scale: float, kh: int = 1, kw: int = 1, stride: int = 1, pad: int = 0,
                 xbar_rows_per_group: Optional[int] = None) -> np.ndarray:
    """grad W = scale * sum_g sum_{j<=K} gamma[g,j] * Eq_j,
    Eq_j = < sum_i B[j,i] delta^(i) , x_bar^(j) >   (Eq. 4, Eq. 6).

    ``xbar`` holds ``xbar_rows_per_group`` encodings per group (K+2 as
    produced by ``encode``, or K+1); only the first K+1 are used.
    """
    G, E, K1 = C.shape
    K = K1 - 1
    rows = E if xbar_rows_per_group is None else xbar_rows_per_group
    delta = np.asarray(delta, dtype=F64)
    xbar = np.asarray(xbar, dtype=F64)
    total = None
    for g in range(G):
        B = derive_B(C[g], gamma[g])
        for j in range(K1):
            dbar = 0.0
            for i in range(K):
                dbar = dbar + B[j, i] * delta[g * K + i]
            eq_j = bilinear_wgrad(dbar, xbar[g * rows + j], kh, kw, stride, pad)
            term = float(gamma[g, j]) * eq_j
            total = term if total is None else total + term
    return scale * total


def wgrad_plain(delta: np.ndarray, x: np.ndarray, scale: float, kh: int = 1, kw: int = 1,
                stride: int = 1, pad: int = 0) -> np.ndarray:
    """grad W = scale * sum_b <delta^(b), x^(b)>  (Eq. 3)."""
    total = None
    for b in range(x.shape[0]):
        t = bilinear_wgrad(delta[b], x[b], kh, kw, stride, pad)
        total = t if total is None else total + t
    return scale * total


def wgrad_plain_at(delta: np.ndarray, x: np.ndarray, scale: float, co: int, ci: int,
                   u: int = 0, v: int = 0, stride: int = 1, pad: int = 0) -> float:
    """One element of ``wgrad_plain`` (only output channel ``co`` of delta and
    input channel ``ci`` of x are converted to float64)."""
    if x.ndim == 2:
        return scale * float(np.asarray(delta[:, co], dtype=F64) @ np.asarray(x[:, ci], dtype=F64))
    d = np.asarray(delta[:, co], dtype=F64)
    _, ho, wo = d.shape
    xp = _pad(np.asarray(x[:, ci:ci + 1], dtype=F64), pad)[:, 0]
    win = xp[:, u:u + (ho - 1) * stride + 1:stride, v:v + (wo - 1) * stride + 1:stride]
    return scale * float(np.sum(d * win))


# ---------------------------------------------------------------------------
# the whole masked forward, step by step
# ---------------------------------------------------------------------------
def masked_forward(W, x, r, C, stride=1, pad=0, tau=1e-4, fault=None, bias=None):
    """encode -> linear on K+2 encodings -> (optional fault) -> decode -> verify.

    ``fault`` = (row of y_bar, index tuple within that row, Delta) models an
    accelerator that returns one wrong value (threat model, Section 3).
    Returns dict with xbar, ybar, y, z and the verify arrays.
    """
    xbar = encode(x, r, C)
    ybar = linear(W, xbar, stride, pad)
    if fault is not None:
        row, idx, dlt = fault
        ybar[(row,) + tuple(idx)] += dlt
    y, z = decode(ybar, C)
    chk = verify(ybar, C, y, z, tau)
    if bias is not None:
        b = np.asarray(bias, dtype=F64)
        y = y + (b if y.ndim == 2 else b[None, :, None, None])
    out = {"xbar": xbar, "ybar": ybar, "y": y, "z": z}
    out.update(chk)
    return out


# ---------------------------------------------------------------------------
# Section 4.4 applied to the weight gradient: two sets of equations
# ---------------------------------------------------------------------------
def second_equation_set(C: np.ndarray, gamma: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Coefficients of the equation set that uses encodings 2..K+2 instead of
    1..K+1: per group the rows of C moved up by one (the first encoding becomes
    the unused last row), and the same for the K+1 gammas (rotated)."""
    C2 = np.concatenate([C[:, 1:], C[:, :1]], axis=1)
    g2 = np.concatenate([gamma[:, 1:], gamma[:, :1]], axis=1)
    return C2, g2


def wgrad_redundant(delta: np.ndarray, xbar: np.ndarray, C: np.ndarray, gamma: np.ndarray,
                    scale: float, kh: int = 1, kw: int = 1, stride: int = 1, pad: int = 0,
                    tau_w: float = 1e-2, fault=None) -> Dict[str, np.ndarray]:
    """grad W decoded twice, from two different sets of K+1 of the K+2 stored
    encodings (Eq. 4-6 with the B of each set), and compared: consistent results
    mean that no term <delta_bar, x_bar^(j)> came back wrong (Section 4.4's
    "computing it redundantly at least twice using at least two sets of
    equations", which the paper states for the forward results only).

    ``xbar`` holds all K+2 encodings per group.  ``fault`` = (which, index
    tuple, value) adds ``value`` to one element of result ``which`` (0 or 1)
    before the comparison.  An element is flagged iff
    not(|dW_0 - dW_1| <= tau_w * rms(dW_0)).
    """
    G, E, K1 = C.shape
    xbar = np.asarray(xbar, dtype=F64)
    first = wgrad_masked(delta, xbar, C, gamma, scale, kh, kw, stride, pad, xbar_rows_per_group=E)
    # the second set: per group encodings 1..K+1, then (unused) encoding 0
    order = np.array([g * E + (i + 1) % E for g in range(G) for i in range(E)])
    C2, g2 = second_equation_set(C, gamma)
    second = wgrad_masked(delta, xbar[order], C2, g2, scale, kh, kw, stride, pad, xbar_rows_per_group=E)
    if fault is not None:
        which, idx, val = fault
        (first if which == 0 else second)[tuple(idx)] += val
    rms = float(np.sqrt(np.mean(first ** 2)))
    diff = np.abs(first - second)
    ratio = diff / rms if rms > 0 else np.where(diff > 0, np.inf, 0.0)
    flags = ~(diff <= tau_w * rms)
    return {"dW": first, "dW_second": second, "ratio": ratio, "flags": flags, "rms": rms}


# ---------------------------------------------------------------------------
# Colluding GPUs (Section 4.5): M noise vectors, S = K + M encodings
# ---------------------------------------------------------------------------
def encode_colluding(x: np.ndarray, R: np.ndarray, A1: np.ndarray, A2: np.ndarray) -> np.ndarray:
    """X_bar = X . A1 + R . A2 for ONE virtual batch (first equation of Section 4.5).

    x: [K, ...] private inputs, R: [M, ...] noise vectors, A1: [K, S], A2: [M, S]
    with S = K + M.  Returns x_bar [S, ...]: encoding j is
    sum_i A1[i, j] x[i] + sum_m A2[m, j] R[m].
    """
    x = np.asarray(x, dtype=np.float64)
    R = np.asarray(R, dtype=np.float64)
    K, M = x.shape[0], R.shape[0]
    S = A1.shape[1]
    assert A1.shape == (K, S) and A2.shape == (M, S) and S == K + M
    out = np.zeros((S,) + x.shape[1:], dtype=np.float64)
    for j in range(S):
        for i in range(K):
            out[j] += A1[i, j] * x[i]
        for m in range(M):
            out[j] += A2[m, j] * R[m]
    return out


def decode_colluding(ybar: np.ndarray, A1: np.ndarray, A2: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Y_bar = [Y | Z] . A with A = [A1; A2] square (S x S): recover Y = <W, X>
    (K results) and Z = <W, R> (M results, dropped by the caller) from the S
    encoded results of one virtual batch, element by element."""
    ybar = np.asarray(ybar, dtype=np.float64)
    A = np.concatenate([A1, A2], axis=0)
    K = A1.shape[0]
    Ainv = invert(A)
    flat = ybar.reshape(ybar.shape[0], -1)            # [S, elements]
    sol = np.zeros_like(flat)
    for u in range(A.shape[0]):                       # unknown u = sum_j ybar[j] * Ainv[j, u]
        for j in range(A.shape[0]):
            sol[u] += Ainv[j, u] * flat[j]
    sol = sol.reshape(ybar.shape)
    return sol[:K], sol[K:]


def colluding_subsets_full_rank(A2: np.ndarray, tol: float = 1e-9) -> bool:
    """The condition Section 5 needs of A2 for M colluders: every choice of M of
    its S columns is a full-rank M x M block, so that no linear combination of
    the encodings a coalition holds is free of noise."""
    import itertools
    M, S = A2.shape
    for cols in itertools.combinations(range(S), M):
        sub = A2[:, cols]
        if np.linalg.matrix_rank(sub, tol=tol) < M:
            return False
    return True


def wgrad_colluding(delta: np.ndarray, xbar: np.ndarray, A1: np.ndarray, A2: np.ndarray,
                    gamma: np.ndarray, scale: float, kh: int = 1, kw: int = 1, stride: int = 1,
                    pad: int = 0) -> np.ndarray:
    """grad W = scale * sum_{j<=S} gamma_j <sum_{i<=K} beta_{j,i} delta^(i), x_bar^(j)> for one
    virtual batch, with B the solution of B^T . Gamma . A = [I_K | 0] (the K x S
    condition of Section 4.5 with A = [A1; A2] as X_bar = [X | R] . A)."""
    A = np.concatenate([A1, A2], axis=0)              # [S, S], rows = sources, columns = encodings
    K, S = A1.shape[0], A.shape[0]
    Ainv = invert(A)
    # B^T Gamma A^T-of-the-sources: with X_bar^T = A^T [X|R]^T the condition reads
    # sum_j B[j,i] gamma_j A[u,j] = [u == i]; hence B[j,i] = Ainv[j,i] / gamma_j
    B = np.zeros((S, K))
    for j in range(S):
        for i in range(K):
            B[j, i] = Ainv[j, i] / gamma[j]
    total = None
    for j in range(S):
        mixed = np.zeros_like(np.asarray(delta[0], dtype=np.float64))
        for i in range(K):
            mixed = mixed + B[j, i] * np.asarray(delta[i], dtype=np.float64)
        eq = bilinear_wgrad(mixed, xbar[j], kh, kw, stride, pad)
        total = gamma[j] * eq if total is None else total + gamma[j] * eq
    return scale * total


# ---------------------------------------------------------------------------
# The unmasked steps around the masked products in a training step: gradient
# back-propagation through a linear layer (Section 4.2: delta_l is computed from
# delta_{l+1} and W "without encoding"), the non-linear layers the paper keeps
# inside the enclave (ReLU, MaxPool; flow of Section 3.1), and the aggregation
# of weight gradients over virtual batches (Section 6, Algorithm 2).
# ---------------------------------------------------------------------------
def dgrad_plain(delta: np.ndarray, W: np.ndarray, in_hw: Tuple[int, int] = (1, 1), stride: int = 1,
                pad: int = 0) -> np.ndarray:
    """Gradient with respect to the layer's input: the adjoint of ``linear``.
    FC: dx = delta @ W.  Convolution: every term W[o,c,u,v] x[n,c,p*s+u-pad,q*s+v-pad] of y[n,o,p,q]
    sends delta[n,o,p,q] W[o,c,u,v] back to that input position."""
    d = np.asarray(delta, dtype=F64)
    W = np.asarray(W, dtype=F64)
    if d.ndim == 2:
        return d @ W
    n, cout, ho, wo = d.shape
    _, cin, kh, kw = W.shape
    h, w = in_hw
    dxp = np.zeros((n, cin, h + 2 * pad, w + 2 * pad), dtype=F64)
    for u in range(kh):
        for v in range(kw):
            # contribution of filter tap (u, v): [n, ho, wo, cin]
            t = np.tensordot(d, W[:, :, u, v], axes=([1], [0])).transpose(0, 3, 1, 2)
            dxp[:, :, u:u + (ho - 1) * stride + 1:stride, v:v + (wo - 1) * stride + 1:stride] += t
    return dxp[:, :, pad:pad + h, pad:pad + w]


def relu(x: np.ndarray) -> np.ndarray:
    return np.maximum(np.asarray(x, dtype=F64), 0.0)


def relu_bwd(dy: np.ndarray, x: np.ndarray) -> np.ndarray:
    """Gradient through ReLU at pre-activation x: passes where x > 0."""
    return np.where(np.asarray(x) > 0, np.asarray(dy, dtype=F64), 0.0)


def maxpool2x2(x: np.ndarray) -> np.ndarray:
    """2x2 max pooling with stride 2 on [n, c, h, w] (h, w even)."""
    x = np.asarray(x, dtype=F64)
    n, c, h, w = x.shape
    win = x.reshape(n, c, h // 2, 2, w // 2, 2)
    return win.max(axis=(3, 5))


def maxpool2x2_bwd(dy: np.ndarray, x: np.ndarray) -> np.ndarray:
    """Gradient through ``maxpool2x2``: each output's gradient goes to the first maximum of its window in
    row-major order (top-left, top-right, bottom-left, bottom-right)."""
    x = np.asarray(x, dtype=F64)
    dy = np.asarray(dy, dtype=F64)
    n, c, h, w = x.shape
    dx = np.zeros_like(x)
    win = x.reshape(n, c, h // 2, 2, w // 2, 2).transpose(0, 1, 2, 4, 3, 5).reshape(n, c, h // 2, w // 2, 4)
    first = np.argmax(win, axis=4)                      # numpy returns the first maximum
    for k in range(4):
        du, dv = divmod(k, 2)
        dx[:, :, du::2, dv::2] = np.where(first == k, dy, 0.0)
    return dx


def training_step_plain(layers, Ws, x0: np.ndarray, dL_dy: np.ndarray, scale: float) -> Dict[str, list]:
    """One training step of a chain of linear layers, each followed by ReLU and optionally a 2x2 max
    pooling, in plain (unmasked) arithmetic: what the masked step must reproduce.

    ``layers``: list of dicts with stride, pad, pool (bool), kh, kw; ``Ws`` their weights; ``x0`` the batch;
    ``dL_dy`` the loss gradient with respect to the last layer's output (after its ReLU/pool).
    Returns the inputs of every layer (``acts``), pre-activations (``pre``), the gradients with respect to
    every pre-activation (``deltas``) and the weight gradients (``dWs``, scaled by ``scale``)."""
    acts, pre = [np.asarray(x0, dtype=F64)], []
    for L, W in zip(layers, Ws):
        z = linear(W, acts[-1], L["stride"], L["pad"])
        pre.append(z)
        a = relu(z)
        acts.append(maxpool2x2(a) if L["pool"] else a)
    g = np.asarray(dL_dy, dtype=F64)
    deltas, dWs = [None] * len(layers), [None] * len(layers)
    for li in range(len(layers) - 1, -1, -1):
        L, W = layers[li], Ws[li]
        if L["pool"]:
            g = maxpool2x2_bwd(g, relu(pre[li]))
        d = relu_bwd(g, pre[li])
        deltas[li] = d
        dWs[li] = wgrad_plain(d, acts[li], scale, L["kh"], L["kw"], L["stride"], L["pad"])
        if li > 0:
            hw = acts[li].shape[2:] if acts[li].ndim == 4 else (1, 1)
            g = dgrad_plain(d, W, hw, L["stride"], L["pad"])
    return {"acts": acts, "pre": pre, "deltas": deltas, "dWs": dWs}
