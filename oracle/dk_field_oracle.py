"""Exact CPU oracle for DarKnight's finite-field arithmetic (Section 5,
"Privacy Guarantee": quantisation, Algorithm 1, coefficients and noise in F_p).

TEST INFRASTRUCTURE ONLY.  Plain and slow; it shares no code with the CUDA
library and must never be imported by it.  Only the tests, the smoke check and
the benchmark's CPU-baseline leg call it.

Everything is integer arithmetic modulo a prime p (the paper uses l = 8
fractional bits and p = 2^25 - 39).  Residues are NumPy int64 arrays in
[0, p); sums of products are reduced often enough that nothing exceeds 2^63
(``_terms_per_reduction``), and the tests pin the results to Python's
unbounded integers.  Logical shapes as in the floating-point oracle: samples
first, then channels, rows, columns.

* ``round_half_up``      procedure Round of Algorithm 1
* ``to_field``           procedure Field of Algorithm 1 (read as
                         ((X mod p) + p) mod p: the printed body is garbled)
* ``quantize``           Field(Round(v * 2^s))
* ``centre``             "subtracts p from all the elements larger than p/2"
* ``dequantize_output``  Round(Y_q * 2^-l) * 2^-l, last step of Algorithm 1
* ``inv_mod`` / ``invert_mod`` / ``null_vector_mod``   small linear algebra in F_p
* ``field_encode``       Eq. 1 (and the redundant encoding of Section 4.4) in F_p
* ``field_linear``       <W_q, x_bar> in F_p (matrix product or cross-correlation)
* ``field_decode``       Eq. 2 in F_p
* ``field_verify``       Section 4.4 with the exact comparison the field allows
* ``field_derive_B`` / ``field_mix_delta`` / ``field_wgrad_masked``
                         Eq. 4-6 in F_p
* ``field_linear_plain`` / ``field_wgrad_plain``   what the masked results must
                         equal, residue for residue (``field_linear_at`` /
                         ``field_wgrad_plain_at``: one element of them, for
                         spot checks on large layers)
* ``field_masked_forward``   procedure Linear Operations of Algorithm 1

Coefficient convention: ``C[g, i, k]`` as in the floating-point oracle (rows
0..K decode, row K+1 is the redundant encoding), entries in [0, p).

Pins (``-m "not gpu"`` tests): a sieve for the prime, hand-derived values of
Round and Field, Fermat's little theorem for the inverse, Python-integer brute
force for every contraction, the encode -> linear -> decode round trip against
the unmasked product, the exact flag set under an injected fault, Eq. 5 in
F_p, the one-time-pad bijection of the privacy lemma on a tiny field, and the
quantisation error bound against the float64 product.
"""
from __future__ import annotations

from typing import Dict, Optional, Tuple

import numpy as np

I64 = np.int64
P_PAPER = 2 ** 25 - 39
L_PAPER = 8


# ---------------------------------------------------------------------------
# the prime
# ---------------------------------------------------------------------------
def is_prime(n: int) -> bool:
    """Trial division."""
    if n < 2:
        return False
    d = 2
    while d * d <= n:
        if n % d == 0:
            return False
        d += 1
    return True


# ---------------------------------------------------------------------------
# Algorithm 1: Round, Field, and the way back
# ---------------------------------------------------------------------------
def round_half_up(v: np.ndarray) -> np.ndarray:
    """Round of Algorithm 1: floor(v) when the fractional part is below one
    half, floor(v) + 1 otherwise.  float64 in, int64 out."""
    v = np.asarray(v, dtype=np.float64)
    f = np.floor(v)
    return np.where(v - f < 0.5, f, f + 1.0).astype(I64)


def to_field(v: np.ndarray, p: int) -> np.ndarray:
    """Field of Algorithm 1: negative values are shifted up by p, then the
    remainder modulo p is taken.  The remainder is taken first as well so that
    one shift suffices for any magnitude."""
    v = np.asarray(v, dtype=I64)
    t = np.fmod(v, I64(p))          # remainder with the sign of v
    t = np.where(t < 0, t + I64(p), t)
    return np.fmod(t, I64(p))


def quantize(v: np.ndarray, scale_bits: int, p: int) -> np.ndarray:
    """Field(Round(v * 2^scale_bits)): scale_bits = l for inputs and weights,
    2l for a bias (Algorithm 1)."""
    return to_field(round_half_up(np.asarray(v, dtype=np.float64) * float(2 ** scale_bits)), p)


def centre(vq: np.ndarray, p: int) -> np.ndarray:
    """Residues above p/2 stand for negative numbers: subtract p from them."""
    vq = np.asarray(vq, dtype=I64)
    return np.where(2 * vq > p, vq - I64(p), vq)


def dequantize_output(yq_centred: np.ndarray, l: int) -> np.ndarray:
    """Y = Round(Y_q * 2^-l) * 2^-l (Y_q carries 2l fractional bits)."""
    r = round_half_up(np.asarray(yq_centred, dtype=np.float64) * float(2.0 ** -l))
    return r.astype(np.float64) * float(2.0 ** -l)


# ---------------------------------------------------------------------------
# small linear algebra in F_p
# ---------------------------------------------------------------------------
def inv_mod(a: int, p: int) -> int:
    """Multiplicative inverse by the extended Euclidean algorithm."""
    a = int(a) % p
    if a == 0:
        raise ZeroDivisionError("0 has no inverse in F_p")
    r0, r1 = p, a
    t0, t1 = 0, 1
    while r1 != 0:
        q = r0 // r1
        r0, r1 = r1, r0 - q * r1
        t0, t1 = t1, t0 - q * t1
    return t0 % p


def invert_mod(M: np.ndarray, p: int) -> np.ndarray:
    """Gauss-Jordan inverse of a small square matrix over F_p (Python ints)."""
    n = M.shape[0]
    a = [[int(M[i, j]) % p for j in range(n)] for i in range(n)]
    inv = [[1 if i == j else 0 for j in range(n)] for i in range(n)]
    for c in range(n):
        piv = next((r for r in range(c, n) if a[r][c] != 0), None)
        if piv is None:
            raise np.linalg.LinAlgError("coefficient block is singular in F_p")
        a[c], a[piv] = a[piv], a[c]
        inv[c], inv[piv] = inv[piv], inv[c]
        ip = inv_mod(a[c][c], p)
        a[c] = [(v * ip) % p for v in a[c]]
        inv[c] = [(v * ip) % p for v in inv[c]]
        for r in range(n):
            if r == c or a[r][c] == 0:
                continue
            f = a[r][c]
            a[r] = [(a[r][j] - f * a[c][j]) % p for j in range(n)]
            inv[r] = [(inv[r][j] - f * inv[c][j]) % p for j in range(n)]
    return np.array(inv, dtype=I64)


def null_vector_mod(Cg: np.ndarray, p: int) -> np.ndarray:
    """n with n^T C = 0 (mod p) and n[K+1] = 1: n[0..K] = -C[K+1] . C_sq^{-1}."""
    K1 = Cg.shape[1]
    inv = invert_mod(Cg[:K1], p)
    n = [(-sum(int(Cg[K1, k]) * int(inv[k, i]) for k in range(K1))) % p for i in range(K1)]
    return np.array(n + [1], dtype=I64)


def _terms_per_reduction(p: int) -> int:
    """How many products of two residues fit into an int64 beside one residue."""
    return max(1, (2 ** 63 - 1 - (p - 1)) // ((p - 1) ** 2))


def _combine(coef, rows, p: int) -> np.ndarray:
    """sum_k coef[k] * rows[k] (mod p), reduced after every term."""
    acc = np.zeros_like(np.asarray(rows[0], dtype=I64))
    for c, row in zip(coef, rows):
        acc = (acc + (I64(int(c)) * np.asarray(row, dtype=I64)) % I64(p)) % I64(p)
    return acc


def _matmul_mod(a: np.ndarray, b: np.ndarray, p: int) -> np.ndarray:
    """a @ b (mod p) for residue matrices, the contraction cut into pieces that
    cannot overflow int64."""
    a = np.asarray(a, dtype=I64)
    b = np.asarray(b, dtype=I64)
    step = _terms_per_reduction(p)
    out = np.zeros((a.shape[0], b.shape[1]), dtype=I64)
    for k0 in range(0, a.shape[1], step):
        out = (out + a[:, k0:k0 + step] @ b[k0:k0 + step]) % I64(p)
    return out


# ---------------------------------------------------------------------------
# Eq. 1 in F_p
# ---------------------------------------------------------------------------
def field_encode(xq: np.ndarray, rq: np.ndarray, Cq: np.ndarray, p: int) -> np.ndarray:
    """x_bar[g*(K+2)+i] = sum_k C[g,i,k] x[g*K+k] + C[g,i,K] r[g]  (mod p)."""
    G, E, K1 = Cq.shape
    K = K1 - 1
    xq = np.asarray(xq, dtype=I64)
    rq = np.asarray(rq, dtype=I64)
    out = np.zeros((G * E,) + xq.shape[1:], dtype=I64)
    for g in range(G):
        for i in range(E):
            out[g * E + i] = _combine(Cq[g, i], [xq[g * K + k] for k in range(K)] + [rq[g]], p)
    return out


# ---------------------------------------------------------------------------
# the bilinear operation in F_p
# ---------------------------------------------------------------------------
def field_linear(Wq: np.ndarray, xq: np.ndarray, p: int, stride: int = 1, pad: int = 0) -> np.ndarray:
    """<W_q, x> per sample modulo p: x @ W^T for 2-D x, else cross-correlation
    with zero padding (0 is the field's zero, so padding commutes with Field)."""
    Wq = np.asarray(Wq, dtype=I64)
    xq = np.asarray(xq, dtype=I64)
    if xq.ndim == 2:
        return _matmul_mod(xq, Wq.T, p)
    n, cin, h, w = xq.shape
    cout, _, kh, kw = Wq.shape
    ho = (h + 2 * pad - kh) // stride + 1
    wo = (w + 2 * pad - kw) // stride + 1
    xp = np.pad(xq, ((0, 0), (0, 0), (pad, pad), (pad, pad)))
    y = np.zeros((n, cout, ho, wo), dtype=I64)
    for u in range(kh):
        for v in range(kw):
            win = xp[:, :, u:u + (ho - 1) * stride + 1:stride, v:v + (wo - 1) * stride + 1:stride]
            rows = win.transpose(0, 2, 3, 1).reshape(-1, cin)              # [(n,p,q), c]
            part = _matmul_mod(rows, Wq[:, :, u, v].T, p)                  # [(n,p,q), o]
            y = (y + part.reshape(n, ho, wo, cout).transpose(0, 3, 1, 2)) % I64(p)
    return y


def field_linear_at(Wq: np.ndarray, x_one: np.ndarray, co: int, oh: int, ow: int, p: int,
                    stride: int = 1, pad: int = 0) -> int:
    """One output element of ``field_linear`` for one sample, in Python integers."""
    if x_one.ndim == 1:
        return sum(int(a) * int(b) for a, b in zip(Wq[co], x_one)) % p
    cin, h, w = x_one.shape
    _, _, kh, kw = Wq.shape
    acc = 0
    for u in range(kh):
        ih = oh * stride + u - pad
        if ih < 0 or ih >= h:
            continue
        for v in range(kw):
            iw = ow * stride + v - pad
            if iw < 0 or iw >= w:
                continue
            acc += sum(int(a) * int(b) for a, b in zip(Wq[co, :, u, v], x_one[:, ih, iw]))
    return acc % p


def field_linear_plain(Wq, xq, p, stride=1, pad=0):
    """What decoding must return: the same operation on the unencoded residues."""
    return field_linear(Wq, xq, p, stride, pad)


# ---------------------------------------------------------------------------
# Eq. 2 and Section 4.4 in F_p
# ---------------------------------------------------------------------------
def field_decode(ybar: np.ndarray, Cq: np.ndarray, p: int) -> Tuple[np.ndarray, np.ndarray]:
    """[y^(1..K); z] = C_sq^{-1} . y_bar^(1..K+1) per group; returns (y, z)."""
    G, E, K1 = Cq.shape
    K = K1 - 1
    ybar = np.asarray(ybar, dtype=I64)
    y = np.zeros((G * K,) + ybar.shape[1:], dtype=I64)
    z = np.zeros((G,) + ybar.shape[1:], dtype=I64)
    for g in range(G):
        inv = invert_mod(Cq[g, :K1], p)
        rows = [ybar[g * E + i] for i in range(K1)]
        for k in range(K):
            y[g * K + k] = _combine(inv[k], rows, p)
        z[g] = _combine(inv[K], rows, p)
    return y, z


def field_verify(ybar: np.ndarray, Cq: np.ndarray, yq: np.ndarray, zq: np.ndarray, p: int) -> np.ndarray:
    """Section 4.4: the redundant equation is predicted from the decoded
    unknowns and compared, exactly, with the value that came back.  Returns the
    flags, one per (group, output element)."""
    G, E, K1 = Cq.shape
    K = K1 - 1
    ybar = np.asarray(ybar, dtype=I64)
    flags = np.zeros((G,) + ybar.shape[1:], dtype=bool)
    for g in range(G):
        pred = _combine(Cq[g, K1], [yq[g * K + k] for k in range(K)] + [zq[g]], p)
        flags[g] = pred != ybar[g * E + K1]
    return flags


def field_verdict(flags: np.ndarray) -> Dict[str, int]:
    """Summary in the order of ``flags.reshape(G, -1)``."""
    flat = flags.reshape(-1)
    idx = np.flatnonzero(flat)
    return {"ok": int(idx.size == 0), "n_flagged": int(idx.size),
            "first_index": int(idx[0]) if idx.size else -1}


# ---------------------------------------------------------------------------
# Eq. 4-6 in F_p
# ---------------------------------------------------------------------------
def field_derive_B(Cg: np.ndarray, gamma_g: np.ndarray, p: int) -> np.ndarray:
    """The B of Eq. 5 for square A = C_sq^T: B[j][i] = (C_sq^{-1})[i][j] / gamma_j."""
    K1 = Cg.shape[1]
    inv = invert_mod(Cg[:K1], p)
    B = np.zeros((K1, K1 - 1), dtype=I64)
    for j in range(K1):
        gi = inv_mod(int(gamma_g[j]), p)
        for i in range(K1 - 1):
            B[j, i] = (int(inv[i, j]) * gi) % p
    return B


def field_mix_delta(deltaq: np.ndarray, B: np.ndarray, g: int, p: int) -> np.ndarray:
    """delta_bar^(j) = sum_i B[j][i] delta^(i) for the K+1 rows j of group g (Eq. 4)."""
    K1, K = B.shape
    return np.stack([_combine(B[j], [deltaq[g * K + i] for i in range(K)], p) for j in range(K1)])


def field_bilinear_wgrad(delta_one: np.ndarray, x_one: np.ndarray, p: int, kh: int = 1, kw: int = 1,
                         stride: int = 1, pad: int = 0) -> np.ndarray:
    """<delta, x> for one sample: outer product, or
    dW[o,c,u,v] = sum_{p,q} delta[o,p,q] x[c,p*stride+u-pad,q*stride+v-pad]."""
    d = np.asarray(delta_one, dtype=I64)
    x = np.asarray(x_one, dtype=I64)
    if x.ndim == 1:
        return _matmul_mod(d[:, None], x[None, :], p)
    cout, ho, wo = d.shape
    cin = x.shape[0]
    xp = np.pad(x, ((0, 0), (pad, pad), (pad, pad)))
    out = np.zeros((cout, cin, kh, kw), dtype=I64)
    for u in range(kh):
        for v in range(kw):
            win = xp[:, u:u + (ho - 1) * stride + 1:stride, v:v + (wo - 1) * stride + 1:stride]
            out[:, :, u, v] = _matmul_mod(d.reshape(cout, -1), win.reshape(cin, -1).T, p)
    return out


def field_wgrad_masked(deltaq: np.ndarray, xbar: np.ndarray, Cq: np.ndarray, gammaq: np.ndarray, p: int,
                       kh: int = 1, kw: int = 1, stride: int = 1, pad: int = 0,
                       xbar_rows: Optional[int] = None) -> np.ndarray:
    """sum_g sum_{j<=K} gamma[g,j] <delta_bar^(j), x_bar^(j)>  (Eq. 4 and 6, summed
    over the virtual batches; the 1/K of Eq. 4 is left to the caller's scale)."""
    G, E, K1 = Cq.shape
    rows = E if xbar_rows is None else xbar_rows
    total = None
    for g in range(G):
        B = field_derive_B(Cq[g], gammaq[g], p)
        dbar = field_mix_delta(deltaq, B, g, p)
        for j in range(K1):
            term = field_bilinear_wgrad(dbar[j], xbar[g * rows + j], p, kh, kw, stride, pad)
            term = (I64(int(gammaq[g, j])) * term) % I64(p)
            total = term if total is None else (total + term) % I64(p)
    return total


def field_wgrad_plain(deltaq: np.ndarray, xq: np.ndarray, p: int, kh: int = 1, kw: int = 1,
                      stride: int = 1, pad: int = 0) -> np.ndarray:
    """sum over samples of <delta^(i), x^(i)> (Eq. 3 without its 1/K)."""
    total = None
    for i in range(xq.shape[0]):
        term = field_bilinear_wgrad(deltaq[i], xq[i], p, kh, kw, stride, pad)
        total = term if total is None else (total + term) % I64(p)
    return total


def field_wgrad_plain_at(deltaq: np.ndarray, xq: np.ndarray, co: int, ci: int, u: int, v: int, p: int,
                         stride: int = 1, pad: int = 0) -> int:
    """One element of ``field_wgrad_plain``, in Python integers."""
    if xq.ndim == 2:
        return sum(int(a) * int(b) for a, b in zip(deltaq[:, co], xq[:, ci])) % p
    n, _, h, w = xq.shape
    _, _, ho, wo = deltaq.shape
    acc = 0
    for a in range(ho):
        ih = a * stride + u - pad
        if ih < 0 or ih >= h:
            continue
        for b in range(wo):
            iw = b * stride + v - pad
            if iw < 0 or iw >= w:
                continue
            acc += sum(int(s) * int(t) for s, t in zip(deltaq[:, co, a, b], xq[:, ci, ih, iw]))
    return acc % p


# ---------------------------------------------------------------------------
# Algorithm 1, procedure Linear Operations
# ---------------------------------------------------------------------------
def field_masked_forward(W, x, rq, Cq, l: int, p: int, stride: int = 1, pad: int = 0, bias=None,
                         fault=None) -> Dict[str, np.ndarray]:
    """Quantise, encode, run the linear operation on the encodings, decode,
    check and return to floating point.  ``rq``: noise residues, one tensor per
    group.  ``bias`` (per output channel) is quantised with 2l bits and added
    after decoding (the masked operation itself is bilinear).  ``fault`` =
    (group, encoding, flat output index, residue added to that element of
    y_bar) models an accelerator that returns one wrong value."""
    Wq = quantize(W, l, p)
    xq = quantize(x, l, p)
    xbar = field_encode(xq, rq, Cq, p)
    ybar = field_linear(Wq, xbar, p, stride, pad)
    if fault is not None:
        g, i, e, d = fault
        E = Cq.shape[1]
        flat = ybar[g * E + i].reshape(-1)
        flat[e] = (flat[e] + int(d)) % p
    yq, zq = field_decode(ybar, Cq, p)
    flags = field_verify(ybar, Cq, yq, zq, p)
    if bias is not None:
        bq = quantize(bias, 2 * l, p)
        shape = (1, -1) + (1,) * (yq.ndim - 2)
        yq = (yq + bq.reshape(shape)) % I64(p)
    yc = centre(yq, p)
    return {"Wq": Wq, "xq": xq, "xbar": xbar, "ybar": ybar, "yq": yc, "y": dequantize_output(yc, l),
            "flags": flags}
