"""Shared helpers of the GPU parity tests: moving seeded inputs to the device
in the library's memory layout, and comparing what comes back with the oracle.
No arithmetic of the method lives here."""
from __future__ import annotations

import numpy as np
import torch

from oracle import dk_oracle as O
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth

TAU = 1e-4


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def acts_to_dev(a: np.ndarray, layout: int) -> torch.Tensor:
    """Logical [n,c,h,w] (or [n,c]) array -> device tensor in `layout`."""
    if a.ndim == 4 and layout == dk.DK_NHWC:
        a = synth.to_channels_last(a)
    return dev(a)


def acts_from_dev(t: torch.Tensor, layout: int) -> np.ndarray:
    a = t.cpu().numpy()
    if a.ndim == 4 and layout == dk.DK_NHWC:
        a = synth.from_channels_last(a)
    return a


def weights_to_dev(W: np.ndarray, layout: int) -> torch.Tensor:
    if W.ndim == 4 and layout == dk.DK_NHWC:
        W = synth.weights_to_ohwi(W)
    return dev(W)


def weights_from_dev(t: torch.Tensor, layout: int) -> np.ndarray:
    W = t.cpu().numpy()
    if W.ndim == 4 and layout == dk.DK_NHWC:
        W = synth.weights_from_ohwi(W)
    return W


def mem_order(a: np.ndarray, layout: int) -> np.ndarray:
    """View of a logical per-sample array in the order the device stores it."""
    if a.ndim == 4 and layout == dk.DK_NHWC:
        return a.transpose(0, 2, 3, 1)
    return a


def empty_acts(n: int, spec, which: str, layout: int) -> torch.Tensor:
    c, h, w = (spec.cin, spec.h, spec.w) if which == "in" else (spec.cout, spec.hout, spec.wout)
    if spec.kind == "fc":
        shape = (n, c)
    elif layout == dk.DK_NHWC:
        shape = (n, h, w, c)
    else:
        shape = (n, c, h, w)
    return torch.empty(shape, dtype=torch.float32, device="cuda")


def empty_weights(spec, layout: int) -> torch.Tensor:
    if spec.kind == "fc":
        shape = (spec.cout, spec.cin)
    elif layout == dk.DK_NHWC:
        shape = (spec.cout, spec.kh, spec.kw, spec.cin)
    else:
        shape = (spec.cout, spec.cin, spec.kh, spec.kw)
    return torch.empty(shape, dtype=torch.float32, device="cuda")


def max_rel(got: np.ndarray, want: np.ndarray) -> float:
    """Max-norm relative error: max|got - want| / max|want|."""
    return float(np.max(np.abs(got.astype(np.float64) - want)) / max(float(np.max(np.abs(want))), 1e-300))


def assert_no_gray_zone(ratio: np.ndarray, tau: float = TAU):
    """A verdict comparison is only meaningful if no element sits near tau."""
    gray = (ratio > tau / 16) & (ratio < tau * 16)
    assert not gray.any(), "oracle ratios fall in the gray zone around tau; redraw the case"


def expected_verdict(flags: np.ndarray, ratio: np.ndarray, layout: int) -> dict:
    return O.verdict(mem_order(flags, layout), mem_order(ratio, layout))


def flat_out_index(spec, layout: int, co: int, oh: int = 0, ow: int = 0) -> int:
    """Index of (co, oh, ow) inside one output sample as stored on the device."""
    if spec.kind == "fc":
        return co
    if layout == dk.DK_NHWC:
        return (oh * spec.wout + ow) * spec.cout + co
    return (co * spec.hout + oh) * spec.wout + ow


def logical_out_index(spec, co: int, oh: int = 0, ow: int = 0):
    return (co,) if spec.kind == "fc" else (co, oh, ow)


def read_positions(spec, a: np.ndarray) -> np.ndarray:
    """The part of a logical input-shaped array [n, c, h, w] that the layer reads: a strided 1x1 convolution
    without padding touches every stride-th row and column only (the library leaves the other positions of
    the stored encodings unwritten); everything else is returned whole."""
    if a.ndim == 4 and spec.kind == "conv" and spec.kh == 1 and spec.kw == 1 and spec.pad == 0 and spec.stride > 1:
        return a[:, :, ::spec.stride, ::spec.stride]
    return a
