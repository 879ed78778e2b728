"""Seeded synthetic workloads for the masked linear-algebra path.

This module only *draws inputs*: layer geometries, private inputs x, noise r,
weights W, output gradients delta, the (K+2)x(K+1) coefficient matrices C and
the diagonal gamma.  It contains none of the method's arithmetic (no encode,
decode, verify or wgrad formula); both the CPU oracle's tests and the CUDA
path's tests/bench take their inputs from here so that the two sides see the
same numbers without sharing any code.

Conventions
-----------
* Logical tensor shapes follow the paper's notation: a virtual batch has K
  private inputs, a batch has G virtual batches (groups) of consecutive
  samples, so ``x`` is ``[G*K, cin, h, w]`` (``[G*K, cin]`` for FC), the noise
  is ``[G, cin, h, w]``, weights are ``[cout, cin, kh, kw]``.
* ``C[g, i, k]`` is the coefficient of source ``k`` (k < K: private input k,
  k = K: the noise) in encoding ``i`` (i < K+1: decodable rows, i = K+1: the
  redundant row used for the integrity check).  In the paper's X_bar = X.A
  notation (Eq. 1) this is ``alpha_{k+1,i+1}``, i.e. C is the transpose of A
  with one more row appended.
* Memory layouts: ``to_channels_last`` / ``weights_to_ohwi`` are pure
  permutations used to hand tensors to the GPU path, which computes
  convolutions on channels-last data.

The real datasets the paper trains on (CIFAR-10, ImageNet) are replaced by
random tensors of the same shapes; layer tables are the usual VGG-16 /
ResNet-18 / MobileNetV2 geometries.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import numpy as np

WORKLOADS = ("fc784", "vgg16_cifar", "resnet18_224", "mobilenetv2_pw", "vgg16_224")

_ROLES = {"x": 1, "r": 2, "w": 3, "delta": 4, "coef": 5, "gamma": 6, "bias": 7, "sample": 8}


@dataclasses.dataclass(frozen=True)
class LayerSpec:
    """Geometry and input statistics of one masked linear layer."""

    workload: str
    name: str
    kind: str            # "fc" or "conv"
    cin: int
    cout: int
    h: int = 1           # input height (1 for fc)
    w: int = 1           # input width
    kh: int = 1
    kw: int = 1
    stride: int = 1
    pad: int = 0
    K: int = 4           # private inputs per virtual batch
    G: int = 1           # virtual batches in the batch
    sigma_r: float = 100.0
    x_dist: str = "uniform"   # "uniform" -> U(0,1), "normal" -> N(0,1)
    w_std: Optional[float] = None   # None -> Kaiming normal sqrt(2/fan_in)
    wgrad: bool = True
    repeat: int = 1      # how many times this shape occurs in the network
    precision: str = "default"   # arithmetic hint for the GPU path: "default" or "fp64"

    @property
    def hout(self) -> int:
        return (self.h + 2 * self.pad - self.kh) // self.stride + 1

    @property
    def wout(self) -> int:
        return (self.w + 2 * self.pad - self.kw) // self.stride + 1

    @property
    def n_in(self) -> int:
        return self.cin * self.h * self.w

    @property
    def n_out(self) -> int:
        return self.cout * self.hout * self.wout

    @property
    def kc(self) -> int:
        return self.cin * self.kh * self.kw

    @property
    def batch(self) -> int:
        return self.K * self.G

    def fwd_flops(self) -> float:
        """Dense flops of the linear op over all K+2 encodings of every group."""
        return 2.0 * self.cout * self.kc * self.G * (self.K + 2) * self.hout * self.wout

    def wgrad_flops(self) -> float:
        """Dense flops of the weight-gradient product over K+1 encodings."""
        return 2.0 * self.cout * self.kc * self.G * (self.K + 1) * self.hout * self.wout

    def with_groups(self, G: int) -> "LayerSpec":
        return dataclasses.replace(self, G=G)


def _conv(workload, name, cin, cout, hw, k=3, s=1, p=None, **kw) -> LayerSpec:
    if p is None:
        p = k // 2
    return LayerSpec(workload, name, "conv", cin, cout, hw, hw, k, k, s, p, **kw)


def _vgg_convs(workload: str, res: int, **kw) -> List[LayerSpec]:
    plan = [("conv1_1", 3, 64, 1), ("conv1_2", 64, 64, 1),
            ("conv2_1", 64, 128, 2), ("conv2_2", 128, 128, 2),
            ("conv3_1", 128, 256, 4), ("conv3_2", 256, 256, 4), ("conv3_3", 256, 256, 4),
            ("conv4_1", 256, 512, 8), ("conv4_2", 512, 512, 8), ("conv4_3", 512, 512, 8),
            ("conv5_1", 512, 512, 16), ("conv5_2", 512, 512, 16), ("conv5_3", 512, 512, 16)]
    return [_conv(workload, n, ci, co, res // d, **kw) for (n, ci, co, d) in plan]


def layers(workload: str) -> List[LayerSpec]:
    """Layer list of one of the five synthetic workloads."""
    if workload == "fc784":
        return [LayerSpec(workload, "fc", "fc", 784, 512, K=2, G=1, sigma_r=100.0,
                          x_dist="uniform", w_std=0.05)]
    if workload == "vgg16_cifar":
        return _vgg_convs(workload, 32, K=4, G=32, sigma_r=100.0, x_dist="uniform")
    if workload == "vgg16_224":
        kw = dict(K=4, G=64, sigma_r=100.0, x_dist="uniform")
        out = _vgg_convs(workload, 224, **kw)
        out += [LayerSpec(workload, "fc6", "fc", 25088, 4096, **kw),
                LayerSpec(workload, "fc7", "fc", 4096, 4096, **kw),
                LayerSpec(workload, "fc8", "fc", 4096, 1000, **kw)]
        return out
    if workload == "resnet18_224":
        kw = dict(K=4, G=16, sigma_r=100.0, x_dist="normal", wgrad=False)
        wl = workload
        return [
            _conv(wl, "stem", 3, 64, 224, k=7, s=2, p=3, **kw),
            _conv(wl, "layer1_3x3", 64, 64, 56, repeat=4, **kw),
            _conv(wl, "layer2_3x3s2", 64, 128, 56, s=2, **kw),
            _conv(wl, "layer2_3x3", 128, 128, 28, repeat=3, **kw),
            _conv(wl, "layer2_ds", 64, 128, 56, k=1, s=2, p=0, **kw),
            _conv(wl, "layer3_3x3s2", 128, 256, 28, s=2, **kw),
            _conv(wl, "layer3_3x3", 256, 256, 14, repeat=3, **kw),
            _conv(wl, "layer3_ds", 128, 256, 28, k=1, s=2, p=0, **kw),
            _conv(wl, "layer4_3x3s2", 256, 512, 14, s=2, **kw),
            _conv(wl, "layer4_3x3", 512, 512, 7, repeat=3, **kw),
            _conv(wl, "layer4_ds", 256, 512, 14, k=1, s=2, p=0, **kw),
            LayerSpec(wl, "fc", "fc", 512, 1000, **kw),
        ]
    if workload == "mobilenetv2_pw":
        # noise 1000x the activations with K = 8: one fp32 rounding of an encoded
        # value is ~1e-4 of the decoded result per unit of decoder gain, so this
        # workload asks the GPU path for its fp64 arithmetic
        kw = dict(K=8, G=16, sigma_r=1000.0, x_dist="normal", wgrad=False, k=1, p=0, precision="fp64")
        wl = workload
        plan = [("expand_16_96", 16, 96, 112), ("project_96_24", 96, 24, 56),
                ("expand_24_144", 24, 144, 56), ("project_144_24", 144, 24, 56),
                ("project_144_32", 144, 32, 28), ("expand_32_192", 32, 192, 28),
                ("project_192_32", 192, 32, 28), ("project_192_64", 192, 64, 14),
                ("expand_64_384", 64, 384, 14), ("project_384_64", 384, 64, 14),
                ("project_384_96", 384, 96, 14), ("expand_96_576", 96, 576, 14),
                ("project_576_96", 576, 96, 14), ("project_576_160", 576, 160, 7),
                ("expand_160_960", 160, 960, 7), ("project_960_160", 960, 160, 7),
                ("project_960_320", 960, 320, 7)]
        return [_conv(wl, n, ci, co, hw, **kw) for (n, ci, co, hw) in plan]
    raise ValueError(f"unknown workload {workload!r}")


def layer(workload: str, name: str) -> LayerSpec:
    for s in layers(workload):
        if s.name == name:
            return s
    raise KeyError(f"{workload}:{name}")


def _rng(spec: LayerSpec, role: str, extra: int = 0) -> np.random.Generator:
    wl = WORKLOADS.index(spec.workload) if spec.workload in WORKLOADS else 99
    names = [s.name for s in layers(spec.workload)] if spec.workload in WORKLOADS else []
    li = names.index(spec.name) if spec.name in names else 999
    return np.random.default_rng(np.random.SeedSequence([2207, 83, wl, li, _ROLES[role], extra]))


# ---------------------------------------------------------------------------
# coefficient matrices
# ---------------------------------------------------------------------------
COND_CAP_PER_DIM = 10.0     # reject C_sq with cond_2 > 10*(K+1)
MIN_NOISE_COEF = 0.1        # every encoding must carry the noise
MIN_NULL_RATIO = 0.05       # every encoding must take part in the redundant equation


def coefficients_acceptable(Cg: np.ndarray) -> bool:
    """Generic linear-algebra screening of one (K+2)x(K+1) coefficient block.

    Uses only library SVDs: the square part must be well conditioned, every
    row must mix in the noise, and the one-dimensional left null space of the
    tall matrix must have no near-zero component (otherwise a fault in that
    encoding would be invisible to any consistency check).
    """
    K1 = Cg.shape[1]
    c64 = Cg.astype(np.float64)
    if np.linalg.cond(c64[:K1]) > COND_CAP_PER_DIM * K1:
        return False
    if np.min(np.abs(c64[:, K1 - 1])) < MIN_NOISE_COEF:
        return False
    u, _, _ = np.linalg.svd(c64, full_matrices=True)
    nv = np.abs(u[:, -1])
    return bool(nv.min() / nv.max() >= MIN_NULL_RATIO)


def draw_coefficients(rng: np.random.Generator, K: int, G: int) -> np.ndarray:
    """iid N(0,1) coefficient blocks, redrawn until ``coefficients_acceptable``."""
    out = np.empty((G, K + 2, K + 1), dtype=np.float32)
    for g in range(G):
        for _ in range(100000):
            cand = rng.standard_normal((K + 2, K + 1)).astype(np.float32)
            if coefficients_acceptable(cand):
                out[g] = cand
                break
        else:  # pragma: no cover
            raise RuntimeError("no acceptable coefficient matrix found")
    return out


def draw_gamma(rng: np.random.Generator, K: int, G: int) -> np.ndarray:
    """gamma_j = +-U(0.5, 2): the secret diagonal of Gamma (Eq. 5)."""
    mag = rng.uniform(0.5, 2.0, size=(G, K + 1))
    sgn = rng.choice([-1.0, 1.0], size=(G, K + 1))
    return (mag * sgn).astype(np.float32)


# ---------------------------------------------------------------------------
# tensors
# ---------------------------------------------------------------------------
def _x_shape(spec: LayerSpec, n: int):
    return (n, spec.cin) if spec.kind == "fc" else (n, spec.cin, spec.h, spec.w)


def _y_shape(spec: LayerSpec, n: int):
    return (n, spec.cout) if spec.kind == "fc" else (n, spec.cout, spec.hout, spec.wout)


def _w_shape(spec: LayerSpec):
    return (spec.cout, spec.cin) if spec.kind == "fc" else (spec.cout, spec.cin, spec.kh, spec.kw)


def draw_layer(spec: LayerSpec, with_delta: bool = True) -> Dict[str, np.ndarray]:
    """All inputs of one layer, float32, logical (channels-first) shapes."""
    rx = _rng(spec, "x")
    if spec.x_dist == "uniform":
        x = rx.random(_x_shape(spec, spec.batch), dtype=np.float32)
    else:
        x = rx.standard_normal(_x_shape(spec, spec.batch), dtype=np.float32)
    r = (_rng(spec, "r").standard_normal(_x_shape(spec, spec.G), dtype=np.float32)
         * np.float32(spec.sigma_r))
    std = spec.w_std if spec.w_std is not None else math.sqrt(2.0 / spec.kc)
    W = _rng(spec, "w").standard_normal(_w_shape(spec), dtype=np.float32) * np.float32(std)
    out = {"x": x, "r": r, "W": W,
           "C": draw_coefficients(_rng(spec, "coef"), spec.K, spec.G),
           "gamma": draw_gamma(_rng(spec, "gamma"), spec.K, spec.G)}
    if with_delta:
        out["delta"] = _rng(spec, "delta").standard_normal(_y_shape(spec, spec.batch), dtype=np.float32)
    return out


def draw_colluding(spec: LayerSpec, K: int, M: int) -> Dict[str, np.ndarray]:
    """Inputs of the M-noise-vector scheme for colluding accelerators (the paper's
    X_bar = X.A1 + R.A2 with S = K + M encodings), laid out so that the library's
    (K_lib + 2) x (K_lib + 1) interface with K_lib = K + M - 1 expresses it:

    * ``x``  [G*K_lib, ...]: per group the K private inputs followed by the first
      M - 1 noise vectors; ``r`` [G, ...]: the M-th noise vector; ``C`` as usual.
    * ``delta`` [G*K_lib, ...]: output gradients of the K private inputs, zeros for
      the rows that stand for noise.
    * the same coefficients and data in the paper's notation: ``A1`` [G, K, S],
      ``A2`` [G, M, S] (rows = sources, columns = encodings, i.e. the transpose of
      the square part of C), ``x_private`` [G, K, ...], ``R`` [G, M, ...],
      ``delta_private`` [G, K, ...].

    Pure relabelling and drawing: nothing of the method is computed here.
    """
    assert spec.K == K + M - 1 and M >= 1
    d = draw_layer(spec, with_delta=True)
    G, KL, S = spec.G, spec.K, K + M
    x = d["x"].reshape((G, KL) + d["x"].shape[1:]).copy()
    if M > 1:
        extra = (_rng(spec, "r", 1).standard_normal((G, M - 1) + x.shape[2:], dtype=np.float32)
                 * np.float32(spec.sigma_r))
        x[:, K:] = extra
    delta = d["delta"].reshape((G, KL) + d["delta"].shape[1:]).copy()
    delta[:, K:] = 0
    A = np.transpose(d["C"][:, :S, :], (0, 2, 1)).astype(np.float64)     # A[g, source, encoding]
    out = dict(d)
    out["x"] = x.reshape(d["x"].shape)
    out["delta"] = delta.reshape(d["delta"].shape)
    out["A1"], out["A2"] = A[:, :K], A[:, K:]
    out["x_private"] = x[:, :K].copy()
    out["R"] = np.concatenate([x[:, K:], d["r"][:, None]], axis=1)
    out["delta_private"] = delta[:, :K].copy()
    return out


def draw_field_layer(spec: LayerSpec, p: int, with_delta: bool = True) -> Dict[str, np.ndarray]:
    """Inputs of one layer for the finite-field arithmetic of the paper's
    Section 5: the same floating-point x, W and delta as ``draw_layer`` plus a
    bias, and what that section draws in the field itself, uniformly: the noise
    ``rq`` [G, ...] over [0, p), the coefficients ``Cq`` [G, K+2, K+1] and the
    diagonal ``gammaq`` [G, K+1] over [1, p).  The coefficient blocks are not
    screened: a singular square part or a vanishing null-space component has
    probability of order K/p.  Quantisation is part of the method and is not
    done here."""
    d = draw_layer(spec, with_delta=with_delta)
    out = {"x": d["x"], "W": d["W"]}
    if with_delta:
        out["delta"] = d["delta"]
    out["bias"] = _rng(spec, "bias").standard_normal(spec.cout, dtype=np.float32) * np.float32(0.1)
    out["rq"] = _rng(spec, "r", 7).integers(0, p, size=_x_shape(spec, spec.G), dtype=np.int64)
    out["Cq"] = _rng(spec, "coef", 7).integers(1, p, size=(spec.G, spec.K + 2, spec.K + 1), dtype=np.int64)
    out["gammaq"] = _rng(spec, "gamma", 7).integers(1, p, size=(spec.G, spec.K + 1), dtype=np.int64)
    return out


def sample_coordinates(spec: LayerSpec, n: int, what: str = "y") -> np.ndarray:
    """Seeded sample of coordinates used for spot checks on large layers.

    ``what="y"``: rows (group, cout, oh, ow), always containing the image
    corners and the last position.  ``what="dw"``: rows (cout, cin, u, v).
    """
    rng = _rng(spec, "sample", 0 if what == "y" else 1)
    if what == "y":
        fixed = [(g, co, oh, ow)
                 for g in (0, spec.G - 1) for co in (0, spec.cout - 1)
                 for oh in (0, spec.hout - 1) for ow in (0, spec.wout - 1)]
        rnd = np.stack([rng.integers(0, spec.G, n), rng.integers(0, spec.cout, n),
                        rng.integers(0, spec.hout, n), rng.integers(0, spec.wout, n)], axis=1)
    else:
        fixed = [(co, ci, u, v) for co in (0, spec.cout - 1) for ci in (0, spec.cin - 1)
                 for u in (0, spec.kh - 1) for v in (0, spec.kw - 1)]
        rnd = np.stack([rng.integers(0, spec.cout, n), rng.integers(0, spec.cin, n),
                        rng.integers(0, spec.kh, n), rng.integers(0, spec.kw, n)], axis=1)
    allc = np.concatenate([np.array(fixed, dtype=np.int64), rnd.astype(np.int64)], axis=0)
    return np.unique(allc, axis=0)


# ---------------------------------------------------------------------------
# pure layout permutations
# ---------------------------------------------------------------------------
def to_channels_last(a: np.ndarray) -> np.ndarray:
    """[n, c, h, w] -> contiguous [n, h, w, c]; 2-D arrays pass through."""
    if a.ndim == 2:
        return np.ascontiguousarray(a)
    return np.ascontiguousarray(a.transpose(0, 2, 3, 1))


def from_channels_last(a: np.ndarray) -> np.ndarray:
    """[n, h, w, c] -> contiguous [n, c, h, w]; 2-D arrays pass through."""
    if a.ndim == 2:
        return np.ascontiguousarray(a)
    return np.ascontiguousarray(a.transpose(0, 3, 1, 2))


def weights_to_ohwi(W: np.ndarray) -> np.ndarray:
    """[cout, cin, kh, kw] -> contiguous [cout, kh, kw, cin]."""
    if W.ndim == 2:
        return np.ascontiguousarray(W)
    return np.ascontiguousarray(W.transpose(0, 2, 3, 1))


def weights_from_ohwi(W: np.ndarray) -> np.ndarray:
    if W.ndim == 2:
        return np.ascontiguousarray(W)
    return np.ascontiguousarray(W.transpose(0, 3, 1, 2))
