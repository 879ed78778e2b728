"""Thin ctypes binding over libdk.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/dk.h).
Tensors are torch CUDA tensors (fp32, contiguous) used purely as device
memory; coefficient matrices are NumPy float32 arrays on the host.  Nothing
here computes: if libdk.so is missing, loading the library fails loudly,
there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdk.so")

DK_FC, DK_CONV2D = 0, 1
DK_NHWC, DK_NCHW = 0, 1
DK_PREC_DEFAULT, DK_TF32X3, DK_FP32_SIMT, DK_FP64_SIMT, DK_TF32X2_WUNSPLIT = 0, 1, 2, 3, 4
(DK_OPT_TC_CHUNK, DK_OPT_WG_CHUNK, DK_OPT_TC_BK, DK_OPT_TC_PAIR, DK_OPT_WG_PACK, DK_OPT_WG_PAIR, DK_OPT_TC_STEM,
 DK_OPT_FIELD_PATH, DK_OPT_SPIN_LIMIT, DK_OPT_TEST_WITHHOLD, DK_OPT_XBAR_HI, DK_OPT_TC_MPACK,
 DK_OPT_SLABS, DK_OPT_SLABS_FORCE, DK_OPT_TC_CHUNK_ADAPT, DK_OPT_WG_PACE, DK_OPT_TC_LO_INKERNEL, DK_OPT_TC_SPLIT_RING, DK_OPT_NOISE_ROWS, DK_OPT_TC_PACE) = range(20)
DK_ERR_TIMEOUT = 6
STATUS_NAMES = ["DK_OK", "DK_ERR_INVALID_ARG", "DK_ERR_SHAPE", "DK_ERR_SINGULAR", "DK_ERR_WORKSPACE",
                "DK_ERR_CUDA", "DK_ERR_TIMEOUT", "DK_ERR_UNSUPPORTED"]


class DkError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where} failed with {name}")


class dk_problem(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("layout", ctypes.c_int32),
                ("cin", ctypes.c_int32), ("cout", ctypes.c_int32),
                ("h", ctypes.c_int32), ("w", ctypes.c_int32),
                ("kh", ctypes.c_int32), ("kw", ctypes.c_int32),
                ("stride", ctypes.c_int32), ("pad", ctypes.c_int32),
                ("K", ctypes.c_int32), ("G", ctypes.c_int32),
                ("precision", ctypes.c_int32), ("tol", ctypes.c_float)]


class dk_verdict(ctypes.Structure):
    _fields_ = [("ok", ctypes.c_int32), ("n_flagged", ctypes.c_uint32),
                ("first_index", ctypes.c_int64), ("max_ratio", ctypes.c_float),
                ("status", ctypes.c_int32)]


class dk_fault(ctypes.Structure):
    _fields_ = [("group", ctypes.c_int32), ("enc", ctypes.c_int32),
                ("out_index", ctypes.c_int64), ("delta", ctypes.c_float)]


class dk_field_fault(ctypes.Structure):
    _fields_ = [("group", ctypes.c_int32), ("enc", ctypes.c_int32),
                ("out_index", ctypes.c_int64), ("delta", ctypes.c_uint32)]


VERDICT_BYTES = ctypes.sizeof(dk_verdict)
_lib = None


def _signatures():
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    pp = ctypes.POINTER(dk_problem)
    return {
        "dk_create": [ctypes.POINTER(vp), ctypes.c_int],
        "dk_destroy": [vp],
        "dk_status_string": [ctypes.c_int],
        "dk_workspace_bytes": [pp, ctypes.POINTER(ctypes.c_size_t)],
        "dk_set_workspace": [vp, vp, ctypes.c_size_t],
        "dk_set_option": [vp, i32, i32],
        "dk_get_option": [vp, i32, ctypes.POINTER(i32)],
        "dk_encode": [vp, pp, vp, vp, vp, vp, vp],
        "dk_linear_fwd": [vp, pp, vp, vp, vp, vp],
        "dk_decode_verify": [vp, pp, vp, vp, vp, vp, vp, vp],
        "dk_masked_linear": [vp, pp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.POINTER(dk_fault), vp],
        "dk_linear_bwd_wgrad": [vp, pp, vp, vp, i32, vp, vp, ctypes.c_float, vp, vp],
        "dk_linear_bwd_wgrad_accumulate": [vp, pp, vp, vp, i32, vp, vp, ctypes.c_float, vp, vp],
        "dk_linear_bwd_dgrad": [vp, pp, vp, vp, vp, vp],
        "dk_relu_pool_fwd": [vp, vp, ctypes.c_int64, i32, i32, i32, i32, vp, vp],
        "dk_relu_pool_bwd": [vp, vp, vp, ctypes.c_int64, i32, i32, i32, i32, vp, vp],
        "dk_linear_bwd_wgrad_verify": [vp, pp, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float, vp, vp,
                                       ctypes.POINTER(dk_fault), vp],
        "dk_decode_verify_static": [ctypes.c_int, pp, vp, vp, vp, vp, vp, vp],
        "dk_device_status": [vp, ctypes.POINTER(ctypes.c_int32)],
        "dk_field_workspace_bytes": [pp, ctypes.POINTER(ctypes.c_size_t)],
        "dk_field_quantize": [vp, vp, ctypes.c_int64, i32, ctypes.c_uint32, vp, vp],
        "dk_field_dequantize": [vp, vp, ctypes.c_int64, i32, ctypes.c_uint32, vp, vp],
        "dk_field_encode": [vp, pp, ctypes.c_uint32, vp, vp, vp, vp, vp],
        "dk_field_linear_fwd": [vp, pp, ctypes.c_uint32, vp, vp, vp, vp],
        "dk_field_decode_verify": [vp, pp, ctypes.c_uint32, i32, vp, vp, vp, vp, vp, vp, vp],
        "dk_field_masked_linear": [vp, pp, ctypes.c_uint32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                   ctypes.POINTER(dk_field_fault), vp],
        "dk_field_linear_bwd_wgrad": [vp, pp, ctypes.c_uint32, vp, vp, i32, vp, vp, vp, vp],
        "dk_profile_enable": [vp, ctypes.c_int],
        "dk_profile_read": [vp, ctypes.c_int, ctypes.POINTER(ctypes.c_double),
                            ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64)],
        "dk_profile_reset": [vp],
    }


EXPORTS = list(_signatures().keys())


def lib() -> ctypes.CDLL:
    """Loads libdk.so (once).  Raises if the library has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2207_00083_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        for name, argtypes in _signatures().items():
            fn = getattr(L, name)
            fn.argtypes = argtypes
            fn.restype = ctypes.c_char_p if name == "dk_status_string" else ctypes.c_int
        _lib = L
    return _lib


def problem_from_spec(spec, layout: int = DK_NHWC, precision: Optional[int] = None,
                      tol: float = 0.0, G: Optional[int] = None) -> dk_problem:
    """dk_problem for a ``synth.LayerSpec``-like object.  ``precision=None``
    follows the spec's own hint (fp64 for the high-noise workload)."""
    kind = DK_FC if spec.kind == "fc" else DK_CONV2D
    if precision is None:
        precision = DK_FP64_SIMT if getattr(spec, "precision", "default") == "fp64" else DK_PREC_DEFAULT
    return dk_problem(kind, layout, spec.cin, spec.cout, spec.h, spec.w, spec.kh, spec.kw,
                      spec.stride, spec.pad, spec.K, spec.G if G is None else G, precision, tol)


def _dev(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise ValueError("expected a contiguous fp32 CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


def _host(a: np.ndarray):
    if not (isinstance(a, np.ndarray) and a.dtype == np.float32 and a.flags["C_CONTIGUOUS"]):
        raise ValueError("expected a C-contiguous float32 NumPy array")
    return ctypes.c_void_p(a.ctypes.data)


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, where: str):
    if status != 0:
        raise DkError(status, where)


class Context:
    """Owns a dk_ctx and (optionally) a torch-allocated workspace."""

    def __init__(self, device: int = 0):
        self._h = ctypes.c_void_p()
        self._ws = None
        torch.cuda.init()
        _check(lib().dk_create(ctypes.byref(self._h), device), "dk_create")
        self.device = device

    def close(self):
        if self._h:
            lib().dk_destroy(self._h)
            self._h = ctypes.c_void_p()
            self._ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self):
        return self._h

    def workspace_bytes(self, p: dk_problem) -> int:
        n = ctypes.c_size_t()
        _check(lib().dk_workspace_bytes(ctypes.byref(p), ctypes.byref(n)), "dk_workspace_bytes")
        return n.value

    def field_workspace_bytes(self, p: dk_problem) -> int:
        n = ctypes.c_size_t()
        _check(lib().dk_field_workspace_bytes(ctypes.byref(p), ctypes.byref(n)), "dk_field_workspace_bytes")
        return n.value

    def ensure_workspace(self, p: dk_problem, field: bool = False):
        """Grows the torch-owned workspace to what `p` needs and registers it
        (``field=True``: what the finite-field calls need)."""
        need = self.field_workspace_bytes(p) if field else self.workspace_bytes(p)
        if self._ws is None or self._ws.numel() < need + 256:
            self._ws = None
            self._ws = torch.empty(need + 256, dtype=torch.uint8, device=f"cuda:{self.device}")
        base = self._ws.data_ptr()
        off = (-base) % 256
        _check(lib().dk_set_workspace(self._h, ctypes.c_void_p(base + off), self._ws.numel() - off),
               "dk_set_workspace")


def dk_set_option(ctx: Context, option: int, value: int):
    _check(lib().dk_set_option(ctx.handle, option, value), "dk_set_option")


def dk_get_option(ctx: Context, option: int) -> int:
    v = ctypes.c_int32()
    _check(lib().dk_get_option(ctx.handle, option, ctypes.byref(v)), "dk_get_option")
    return v.value


KERNEL_KINDS = ["encode", "linear_fwd", "decode_verify", "mix_delta", "wgrad", "other"]


def dk_profile_enable(ctx: Context, on: bool):
    _check(lib().dk_profile_enable(ctx.handle, int(on)), "dk_profile_enable")


def dk_profile_reset(ctx: Context):
    _check(lib().dk_profile_reset(ctx.handle), "dk_profile_reset")


def dk_profile_read(ctx: Context) -> dict:
    """{kind: (ms_total, timed_launches, all_launches)} since the last reset."""
    out = {}
    for k, name in enumerate(KERNEL_KINDS):
        ms, nt, na = ctypes.c_double(), ctypes.c_int64(), ctypes.c_int64()
        _check(lib().dk_profile_read(ctx.handle, k, ctypes.byref(ms), ctypes.byref(nt), ctypes.byref(na)),
               "dk_profile_read")
        out[name] = (ms.value, nt.value, na.value)
    return out


def new_verdict(device: int = 0) -> torch.Tensor:
    """Device storage for one dk_verdict."""
    return torch.zeros(VERDICT_BYTES, dtype=torch.uint8, device=f"cuda:{device}")


def read_verdict(v: torch.Tensor) -> dict:
    """Synchronising device->host read of a dk_verdict."""
    raw = v.cpu().numpy().tobytes()
    s = dk_verdict.from_buffer_copy(raw)
    return {"ok": int(s.ok), "n_flagged": int(s.n_flagged), "first_index": int(s.first_index),
            "max_ratio": float(s.max_ratio), "status": int(s.status)}


def dk_encode(ctx: Context, p: dk_problem, x, r, C: np.ndarray, xbar):
    _check(lib().dk_encode(ctx.handle, ctypes.byref(p), _dev(x), _dev(r), _host(C), _dev(xbar), _stream()),
           "dk_encode")


def dk_linear_fwd(ctx: Context, p: dk_problem, W, xbar, ybar):
    _check(lib().dk_linear_fwd(ctx.handle, ctypes.byref(p), _dev(W), _dev(xbar), _dev(ybar), _stream()),
           "dk_linear_fwd")


def dk_decode_verify(ctx: Context, p: dk_problem, ybar, C: np.ndarray, bias, y, verdict):
    _check(lib().dk_decode_verify(ctx.handle, ctypes.byref(p), _dev(ybar), _host(C), _dev(bias), _dev(y),
                                  ctypes.c_void_p(verdict.data_ptr()), _stream()), "dk_decode_verify")


def dk_decode_verify_static(device: int, p: dk_problem, ybar, C: np.ndarray, bias, y, verdict):
    """Same result as dk_decode_verify, for callers that may not allocate: no
    context, scratch in a fixed array inside the library (see include/dk.h)."""
    _check(lib().dk_decode_verify_static(device, ctypes.byref(p), _dev(ybar), _host(C), _dev(bias), _dev(y),
                                         ctypes.c_void_p(verdict.data_ptr()), _stream()),
           "dk_decode_verify_static")


def dk_device_status(ctx: Context) -> int:
    """Synchronises and returns (then clears) the status raised on the device by
    calls that have no verdict (0 = none)."""
    v = ctypes.c_int32()
    _check(lib().dk_device_status(ctx.handle, ctypes.byref(v)), "dk_device_status")
    return v.value


def dk_masked_linear(ctx: Context, p: dk_problem, W, x, r, C: np.ndarray, bias, y, xbar_save, verdict,
                     fault: Optional[dk_fault] = None):
    fp = ctypes.byref(fault) if fault is not None else None
    _check(lib().dk_masked_linear(ctx.handle, ctypes.byref(p), _dev(W), _dev(x), _dev(r), _host(C),
                                  _dev(bias), _dev(y), _dev(xbar_save),
                                  ctypes.c_void_p(verdict.data_ptr()), fp, _stream()), "dk_masked_linear")


def dk_linear_bwd_wgrad_verify(ctx: Context, p: dk_problem, delta, xbar, C: np.ndarray, gamma: np.ndarray,
                               scale: float, tol_w: float, dW, verdict, fault=None):
    fp = ctypes.byref(fault) if fault is not None else None
    _check(lib().dk_linear_bwd_wgrad_verify(ctx.handle, ctypes.byref(p), _dev(delta), _dev(xbar), _host(C),
                                            _host(gamma), ctypes.c_float(scale), ctypes.c_float(tol_w), _dev(dW),
                                            ctypes.c_void_p(verdict.data_ptr()), fp, _stream()),
           "dk_linear_bwd_wgrad_verify")


def dk_linear_bwd_wgrad(ctx: Context, p: dk_problem, delta, xbar, xbar_rows: int, C: np.ndarray,
                        gamma: np.ndarray, scale: float, dW):
    _check(lib().dk_linear_bwd_wgrad(ctx.handle, ctypes.byref(p), _dev(delta), _dev(xbar), xbar_rows,
                                     _host(C), _host(gamma), ctypes.c_float(scale), _dev(dW), _stream()),
           "dk_linear_bwd_wgrad")


def dk_linear_bwd_wgrad_accumulate(ctx: Context, p: dk_problem, delta, xbar, xbar_rows: int, C: np.ndarray,
                                   gamma: np.ndarray, scale: float, dW):
    _check(lib().dk_linear_bwd_wgrad_accumulate(ctx.handle, ctypes.byref(p), _dev(delta), _dev(xbar), xbar_rows,
                                                _host(C), _host(gamma), ctypes.c_float(scale), _dev(dW),
                                                _stream()), "dk_linear_bwd_wgrad_accumulate")


def dk_linear_bwd_dgrad(ctx: Context, p: dk_problem, W, delta, dx):
    _check(lib().dk_linear_bwd_dgrad(ctx.handle, ctypes.byref(p), _dev(W), _dev(delta), _dev(dx), _stream()),
           "dk_linear_bwd_dgrad")


def dk_relu_pool_fwd(ctx: Context, x, n: int, h: int, w: int, c: int, pool: bool, y):
    _check(lib().dk_relu_pool_fwd(ctx.handle, _dev(x), n, h, w, c, int(pool), _dev(y), _stream()),
           "dk_relu_pool_fwd")


def dk_relu_pool_bwd(ctx: Context, dy, x, n: int, h: int, w: int, c: int, pool: bool, dx):
    _check(lib().dk_relu_pool_bwd(ctx.handle, _dev(dy), _dev(x), n, h, w, c, int(pool), _dev(dx), _stream()),
           "dk_relu_pool_bwd")


# ---------------------------------------------------------------------------
# finite-field calls: residues are int32 CUDA tensors holding values in [0, p)
# (the library reads them as uint32), coefficient arrays NumPy uint32 on the host
# ---------------------------------------------------------------------------
def _res(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not (t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()):
        raise ValueError("expected a contiguous int32 CUDA tensor of residues")
    return ctypes.c_void_p(t.data_ptr())


def _host_u32(a: np.ndarray):
    if not (isinstance(a, np.ndarray) and a.dtype == np.uint32 and a.flags["C_CONTIGUOUS"]):
        raise ValueError("expected a C-contiguous uint32 NumPy array")
    return ctypes.c_void_p(a.ctypes.data)


def dk_field_quantize(ctx: Context, v, scale_bits: int, prime: int, vq):
    _check(lib().dk_field_quantize(ctx.handle, _dev(v), v.numel(), scale_bits, prime, _res(vq), _stream()),
           "dk_field_quantize")


def dk_field_dequantize(ctx: Context, vq, scale_bits: int, prime: int, v):
    _check(lib().dk_field_dequantize(ctx.handle, _res(vq), vq.numel(), scale_bits, prime, _dev(v), _stream()),
           "dk_field_dequantize")


def dk_field_encode(ctx: Context, p: dk_problem, prime: int, xq, rq, C: np.ndarray, xbar):
    _check(lib().dk_field_encode(ctx.handle, ctypes.byref(p), prime, _res(xq), _res(rq), _host_u32(C),
                                 _res(xbar), _stream()), "dk_field_encode")


def dk_field_linear_fwd(ctx: Context, p: dk_problem, prime: int, Wq, xbar, ybar):
    _check(lib().dk_field_linear_fwd(ctx.handle, ctypes.byref(p), prime, _res(Wq), _res(xbar), _res(ybar),
                                     _stream()), "dk_field_linear_fwd")


def dk_field_decode_verify(ctx: Context, p: dk_problem, prime: int, l: int, ybar, C: np.ndarray, bias_q, yq, y,
                           verdict):
    _check(lib().dk_field_decode_verify(ctx.handle, ctypes.byref(p), prime, l, _res(ybar), _host_u32(C),
                                        _res(bias_q), _res(yq), _dev(y), ctypes.c_void_p(verdict.data_ptr()),
                                        _stream()), "dk_field_decode_verify")


def dk_field_masked_linear(ctx: Context, p: dk_problem, prime: int, l: int, W, x, rq, C: np.ndarray, bias, y, yq,
                           xbar_save, verdict, fault: Optional[dk_field_fault] = None):
    fp = ctypes.byref(fault) if fault is not None else None
    _check(lib().dk_field_masked_linear(ctx.handle, ctypes.byref(p), prime, l, _dev(W), _dev(x), _res(rq),
                                        _host_u32(C), _dev(bias), _dev(y), _res(yq), _res(xbar_save),
                                        ctypes.c_void_p(verdict.data_ptr()), fp, _stream()),
           "dk_field_masked_linear")


def dk_field_linear_bwd_wgrad(ctx: Context, p: dk_problem, prime: int, deltaq, xbar, xbar_rows: int, C: np.ndarray,
                              gamma: np.ndarray, dWq):
    _check(lib().dk_field_linear_bwd_wgrad(ctx.handle, ctypes.byref(p), prime, _res(deltaq), _res(xbar), xbar_rows,
                                           _host_u32(C), _host_u32(gamma), _res(dWq), _stream()),
           "dk_field_linear_bwd_wgrad")
