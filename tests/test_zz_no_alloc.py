"""dk_decode_verify_static: the decode + integrity check for callers that may
not allocate device memory (fixed memory budgets, sections that cannot take
the device-wide synchronisation of an allocation, processes that must not
create a context).  Its scratch is a fixed array inside the library, shared by
all calls, so the test makes two calls in a row (the second on different data,
with one wrong accelerator output) and compares each with what the ordinary
entry point dk_decode_verify returns for the same inputs.

Collected last on purpose: a run that stops at the first failure has already
run every other test."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import dk_oracle as O
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu

TOL_DECODED = 1e-3


def _inputs(spec):
    d = synth.draw_layer(spec)
    ybar = O.linear(d["W"], O.encode(d["x"], d["r"], d["C"]), spec.stride, spec.pad).astype(np.float32)
    return d, ybar


def _both(ctx, spec, p, ybar, C, bias):
    """Runs the ordinary and the allocation-free entry point on the same inputs."""
    yb = H.acts_to_dev(ybar, dk.DK_NHWC)
    b = None if bias is None else H.dev(bias)
    y_ref = H.empty_acts(spec.batch, spec, "out", dk.DK_NHWC)
    y_new = torch.full_like(y_ref, float("nan"))
    v_ref, v_new = dk.new_verdict(), dk.new_verdict()
    dk.dk_decode_verify(ctx, p, yb, C, b, y_ref, v_ref)
    dk.dk_decode_verify_static(0, p, yb, C, b, y_new, v_new)
    return y_ref, dk.read_verdict(v_ref), y_new, dk.read_verdict(v_new)


def test_static_entry_point_matches_decode_verify_twice_in_a_row():
    spec = synth.layer("vgg16_cifar", "conv4_1").with_groups(3)
    p = dk.problem_from_spec(spec, tol=H.TAU)
    d, ybar = _inputs(spec)
    bias = np.linspace(-2.0, 2.0, spec.cout).astype(np.float32)
    ctx = dk.Context(0)
    try:
        # first call: clean run
        y_ref, v_ref, y_new, v_new = _both(ctx, spec, p, ybar, d["C"], bias)
        # the group rms behind max_ratio is summed with fp32 atomics: last bits may differ
        assert v_new["max_ratio"] == pytest.approx(v_ref["max_ratio"], rel=1e-5)
        assert (v_new["ok"], v_new["n_flagged"], v_new["first_index"], v_new["status"]) == \
               (v_ref["ok"], v_ref["n_flagged"], v_ref["first_index"], v_ref["status"]) == (1, 0, -1, 0)
        got, want = y_new.cpu().numpy().astype(np.float64), y_ref.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(got - want)) <= TOL_DECODED * np.max(np.abs(want))
        yd, _ = O.decode(ybar, d["C"])
        assert H.max_rel(H.acts_from_dev(y_new, dk.DK_NHWC), yd + bias[None, :, None, None]) < TOL_DECODED

        # second call straight after, other data: two wrong values in different groups
        bad = ybar.copy()
        E = spec.K + 2
        rms = float(np.sqrt(np.mean(bad.astype(np.float64) ** 2)))
        bad[1 * E + 2, 7, 1, 3] += np.float32(0.5 * rms)
        bad[2 * E + 5, 500, 3, 0] -= np.float32(0.5 * rms)
        y_ref, v_ref, y_new, v_new = _both(ctx, spec, p, bad, d["C"], None)
        assert v_new["status"] == 0
        assert (v_new["ok"], v_new["n_flagged"], v_new["first_index"]) == \
               (v_ref["ok"], v_ref["n_flagged"], v_ref["first_index"]) == \
               (0, 2, 1 * spec.n_out + H.flat_out_index(spec, dk.DK_NHWC, 7, 1, 3))
        assert v_new["max_ratio"] == pytest.approx(v_ref["max_ratio"], rel=1e-5)
        got, want = y_new.cpu().numpy().astype(np.float64), y_ref.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(got - want)) <= TOL_DECODED * np.max(np.abs(want))

        # third call: clean again, nothing of the faulted call may linger
        _, _, y_new, v_new = _both(ctx, spec, p, ybar, d["C"], bias)
        assert (v_new["ok"], v_new["n_flagged"], v_new["first_index"]) == (1, 0, -1)
    finally:
        ctx.close()


def test_static_entry_point_leaves_free_device_memory_unchanged():
    """What the call exists for: with no context alive, a warmed-up call must not change the amount of
    free device memory (no allocation by the call itself or by anything it uses)."""
    spec = synth.layer("vgg16_cifar", "conv4_1").with_groups(2)
    p = dk.problem_from_spec(spec, tol=H.TAU)
    d, ybar = _inputs(spec)
    yb = H.acts_to_dev(ybar, dk.DK_NHWC)
    y = H.empty_acts(spec.batch, spec, "out", dk.DK_NHWC)
    v = dk.new_verdict()
    dk.dk_decode_verify_static(0, p, yb, d["C"], None, y, v)      # first call on the device: address look-up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        dk.dk_decode_verify_static(0, p, yb, d["C"], None, y, v)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert dk.read_verdict(v)["ok"] == 1


def test_static_entry_point_refuses_a_capturing_stream():
    """The tables are copied from the call's stack frame, so a call on a capturing stream is refused."""
    spec = synth.layer("vgg16_cifar", "conv5_1").with_groups(1)
    p = dk.problem_from_spec(spec, tol=H.TAU)
    d, ybar = _inputs(spec)
    yb = H.acts_to_dev(ybar, dk.DK_NHWC)
    y = H.empty_acts(spec.batch, spec, "out", dk.DK_NHWC)
    v = dk.new_verdict()
    dk.dk_decode_verify_static(0, p, yb, d["C"], None, y, v)
    torch.cuda.synchronize()
    C = np.ascontiguousarray(d["C"], dtype=np.float32)
    st = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        graph.capture_begin()
        rc = dk.lib().dk_decode_verify_static(0, ctypes.byref(p), ctypes.c_void_p(yb.data_ptr()),
                                              ctypes.c_void_p(C.ctypes.data), None, ctypes.c_void_p(y.data_ptr()),
                                              ctypes.c_void_p(v.data_ptr()), ctypes.c_void_p(st.cuda_stream))
        graph.capture_end()
    assert rc == 7      # DK_ERR_UNSUPPORTED, nothing recorded
    dk.dk_decode_verify_static(0, p, yb, d["C"], None, y, v)      # and the entry point still works afterwards
    assert dk.read_verdict(v)["ok"] == 1


def test_static_entry_point_refuses_what_does_not_fit():
    spec = synth.LayerSpec("tiny", "t", "fc", 16, 8, K=8, G=400)      # tables beyond the fixed array
    p = dk.problem_from_spec(spec)
    t = torch.zeros(16, device="cuda")
    C = np.zeros((400, 10, 9), dtype=np.float32)
    rc = dk.lib().dk_decode_verify_static(0, ctypes.byref(p), ctypes.c_void_p(t.data_ptr()),
                                          ctypes.c_void_p(C.ctypes.data), None,
                                          ctypes.c_void_p(t.data_ptr()), ctypes.c_void_p(t.data_ptr()), None)
    assert rc == 4      # DK_ERR_WORKSPACE, nothing launched
