#!/usr/bin/env python
"""Benchmark of the masked linear-algebra path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload vgg16_224] [--no-cpu-baseline] [--no-field]
    python bench.py --layer-table [--workload vgg16_224] [--layers conv3_2,conv4_2]
    python bench.py --field-table [--workload vgg16_cifar] [--layers conv3_2,conv4_2]
    python bench.py --schedule [--workload vgg16_224]

One step = one pass of the whole path over one synthetic batch of the
workload: for every layer the fused masked forward (encode, dense op on the
K+2 encodings, decode, integrity check, with the encodings stored) followed by
the masked weight gradient where the workload trains.  Prints ONE JSON line.

The default workload is the full VGG-16 step at 224 x 224, batch 256 (13
convolutions and 3 fully connected layers, all resident).  Beside the step
metric the line carries, per layer and call, the roof that binds it (tensor
or HBM) and the fraction reached; the ten-step schedule with one injected
wrong accelerator output and what the integrity check said; and the smallest
wrong value the floating-point check flags, measured through the C-ABI.

`--impl reference` times the fp64 CPU oracle as it stands on a bounded sample
of the same workload (step i = one virtual batch of layer i mod L).

`--layer-table` times every layer of a workload on its own (forward call and
wgrad call, CUDA events around the C-ABI call) and prints one JSON line with
the per-layer table; it is a reporting aid, not the step metric.

`--field-table` does the same for the finite-field calls (Section 5 of the
paper: residues modulo p = 2^25 - 39), in exact modular multiply-accumulates
per second against the peak of the integer tensor pipe they run on.

With N > 1 (under torchrun) every rank runs an independent replica of the
workload on its own GPU: the path has no exchange step, nothing is sharded.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "decoded masked-linear TFLOP/s & fraction of roofline; encode/decode GB/s"
L2_FLUSH_BYTES = 512 << 20
TF32_OVER_BF16 = 1.1 / 2.25      # nominal dense TF32 : BF16 tensor throughput
FP32_ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # SMs x FMA lanes x 2 x max SM clock
# fp64 rate of this part: 148 SMs x 64 fp64 FMA lanes x 2 x 1.965 GHz = 37.2 TFLOP/s; a register-resident loop of
# mma.sync.m8n8k4.f64 measured 37.0 and one of plain fp64 FMAs 36.6 on this machine
FP64_PEAK_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12
# DRAM bytes (read + write) of all launches of a GEMM kernel class in ONE step of the workload, from ncu captures
# of these kernels (summaries with their commands under profiles/); the bench line divides by the launches per
# step.  A workload or class that is absent here has not been captured since the kernels last changed and
# reports null.
NCU_TRAFFIC_BYTES_PER_STEP = {"vgg16_224": {"linear_fwd": 45109597952, "wgrad": 69636159232}}


def apply_options(dk, ctx, args):
    """--option NAME=VALUE pairs -> dk_set_option; returns them as a dict for the output line."""
    out = {}
    for item in args.option:
        name, value = item.split("=", 1)
        dk.dk_set_option(ctx, getattr(dk, "DK_OPT_" + name.upper()), int(value))
        out[name.upper()] = int(value)
    return out


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ---------------------------------------------------------------------------
# reference arm / CPU baseline: the oracle on one virtual batch of every layer
# ---------------------------------------------------------------------------
def oracle_layer_sample(spec, d):
    """The oracle's masked forward (+ check, + masked wgrad where the workload trains) on ONE virtual batch
    (G = 1) of one layer.  Returns the masked flops it covered."""
    from oracle import dk_oracle as O
    m = O.masked_forward(d["W"], d["x"], d["r"], d["C"], spec.stride, spec.pad)
    flops = spec.fwd_flops()
    if spec.wgrad:
        O.wgrad_masked(d["delta"], m["xbar"], d["C"], d["gamma"], 1.0 / spec.batch,
                       spec.kh, spec.kw, spec.stride, spec.pad)
        flops += spec.wgrad_flops()
    return flops


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def time_oracle(workload, steps, warmup, budget_s=None):
    """Times the oracle as it stands on a bounded sample of the workload: step i runs one virtual batch
    (G = 1) of layer (i mod L) of the workload's L layers, so that L consecutive steps cover one group of
    every layer; with `budget_s` the run stops at the first step boundary past the budget."""
    from paper_2207_00083_b200 import synth
    specs = [s.with_groups(1) for s in synth.layers(workload)]
    n = len(specs)
    drawn = {}

    def one(i):
        li = i % n
        if li not in drawn:
            drawn[li] = synth.draw_layer(specs[li], with_delta=specs[li].wgrad)
        return oracle_layer_sample(specs[li], drawn[li])

    for i in range(warmup):
        one(i)
    for i in range(warmup, warmup + steps):      # inputs are drawn outside the timed region
        li = i % n
        if li not in drawn:
            drawn[li] = synth.draw_layer(specs[li], with_delta=specs[li].wgrad)
    flops, done, dt = 0.0, 0, 0.0
    for i in range(warmup, warmup + steps):
        t0 = time.perf_counter()
        flops += one(i)
        dt += time.perf_counter() - t0
        done += 1
        if budget_s is not None and dt > budget_s:
            break
    covered = [specs[i % n].name for i in range(warmup, warmup + done)]
    return {"value": flops / dt / 1e12, "ms_per_step": dt / done * 1e3, "steps": done,
            "sample": f"{done} steps, step i = one virtual batch (G=1) of layer (i mod {n}) of {workload}: masked "
                      f"forward+verify" + (" and masked wgrad" if specs[0].wgrad else "") +
                      f"; layers covered: {','.join(covered)}",
            "cores": cpu_threads()}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    r = time_oracle(args.workload, max(1, args.steps), max(0, args.warmup))
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": "TFLOP/s",
            "n_gpus": args.gpus, "steps": r["steps"], "warmup": args.warmup, "ms_per_step": r["ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": args.workload, "sample": r["sample"]},
            "cpu_baseline": {"value": r["value"], "unit": "TFLOP/s", "cores": r["cores"], "kind": "oracle",
                             "sample": r["sample"]},
            "e2e": {"value": r["value"], "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# helpers of our arm
# ---------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.QUERY}",
                                       "--format=csv,noheader,nounits", "-lms", "50"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
            time.sleep(0.3)      # let the sampler come up before the timed region
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except Exception:
                self.p.kill()
        try:
            self.f.flush()
            self.f.seek(0)
            sm, mx, reasons = [], [], set()
            for ln in self.f:
                c = [t.strip() for t in ln.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1])); mx.append(float(c[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), c[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            if sm:
                out = {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)),
                       "reasons": sorted(reasons), "samples": len(sm)}
        finally:
            self.f.close()
            os.unlink(self.f.name)
        return out


def shape_acts(n, s, which):
    c, h, w = (s.cin, s.h, s.w) if which == "in" else (s.cout, s.hout, s.wout)
    return (n, c) if s.kind == "fc" else (n, h, w, c)


def shape_w(s):
    return (s.cout, s.cin) if s.kind == "fc" else (s.cout, s.kh, s.kw, s.cin)


def uses_tensor_cores(s):
    """Mirror of the library's dispatch rule (channels-last, default arithmetic; stride <= 4 and
    cin % 4 == 0, or a stem whose contraction has 65..256 elements: cin % 4 != 0 laid out as patch rows;
    stems of 1-3 channels with at most 64 elements run in the fused fp32 kernel)."""
    if getattr(s, "precision", "default") != "default":
        return False
    if s.cin % 4 == 0:
        return s.stride <= 4
    if s.cin <= 3 and s.kc <= 64:
        return False
    return s.kind == "conv" and s.kc <= 256 and s.cout % 4 == 0


def make_layer(torch, dk, synth, ctx, s, dev, gen, rank, pinned):
    """Device tensors of one layer, seeded (`pinned` is unused: host copies are made by measure_e2e)."""
    p = dk.problem_from_spec(s, tol=1e-4)
    rng = synth._rng(s, "coef", rank)
    L = {"spec": s, "p": p, "C": synth.draw_coefficients(rng, s.K, s.G),
         "gamma": synth.draw_gamma(rng, s.K, s.G)}
    x = torch.empty(shape_acts(s.batch, s, "in"), device=dev)
    if s.x_dist == "uniform":
        x.uniform_(0, 1, generator=gen)
    else:
        x.normal_(0, 1, generator=gen)
    r = torch.empty(shape_acts(s.G, s, "in"), device=dev).normal_(0, s.sigma_r, generator=gen)
    std = s.w_std if s.w_std is not None else (2.0 / s.kc) ** 0.5
    L["x"], L["r"] = x, r
    L["W"] = torch.randn(shape_w(s), device=dev, generator=gen) * std
    L["y"] = torch.empty(shape_acts(s.batch, s, "out"), device=dev)
    L["xsave"] = torch.empty(shape_acts(s.G * (s.K + 2), s, "in"), device=dev)
    L["v"] = dk.new_verdict(dev.index)
    if s.wgrad:
        L["delta"] = torch.empty(shape_acts(s.batch, s, "out"), device=dev).normal_(0, 1, generator=gen)
        L["dW"] = torch.empty_like(L["W"])
    return L


def measure_elementwise(torch, dk, synth, ctx, dev, peaks, iters=10):
    """Standalone dk_encode / dk_decode_verify on tensors much larger than L2."""
    K, G, n = 4, 32, 1 << 20
    spec = synth.LayerSpec("elementwise", "stream", "fc", n, n, K=K, G=G)
    p = dk.problem_from_spec(spec, tol=1e-4)
    rng = np.random.default_rng(7)
    C = synth.draw_coefficients(rng, K, G)
    x = torch.rand((G * K, n), device=dev)
    r = torch.randn((G, n), device=dev) * 100.0
    xbar = torch.empty((G * (K + 2), n), device=dev)
    y = torch.empty((G * K, n), device=dev)
    v = dk.new_verdict(dev.index)
    out = {}
    for name, fn, bytes_per_pos in (
            ("encode", lambda: dk.dk_encode(ctx, p, x, r, C, xbar), (2 * K + 3) * 4),
            ("decode", lambda: dk.dk_decode_verify(ctx, p, xbar, C, None, y, v), (2 * K + 2) * 4)):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / iters
        gbs = bytes_per_pos * G * n / (ms * 1e-3) / 1e9
        out[name] = {"gbs": gbs, "frac_hbm": gbs / peaks["hbm_gbs"], "ms": ms,
                     "bytes": bytes_per_pos * G * n, "shape": f"K={K} G={G} n={n} fp32"}
    assert dk.read_verdict(v)["status"] == 0
    return out


def run_layer_table(args):
    """Every layer of a workload on its own (one layer resident at a time): see profile_layers."""
    import torch
    from paper_2207_00083_b200 import binding as dk
    from paper_2207_00083_b200 import synth
    dev = torch.device("cuda:0")
    torch.cuda.set_device(0)
    peaks = read_peaks()
    tf32_peak = peaks["bf16_tflops"] * TF32_OVER_BF16
    ctx = dk.Context(0)
    options = apply_options(dk, ctx, args)
    gen = torch.Generator(device=dev)
    gen.manual_seed(220700083)
    flush = torch.empty(L2_FLUSH_BYTES // 4, dtype=torch.float32, device=dev)
    want = set(args.layers.split(",")) if args.layers else None
    rows = []
    for s in synth.layers(args.workload):
        if want and s.name not in want:
            continue
        if args.groups > 0:
            s = s.with_groups(args.groups)      # a smaller batch of the same layer (for profiler captures)
        L = make_layer(torch, dk, synth, ctx, s, dev, gen, 0, pinned=False)
        ctx.ensure_workspace(L["p"])
        row = profile_layers(torch, dk, ctx, [L], peaks, tf32_peak, flush, iters=args.iters)[0]
        row["verdict_ok"] = dk.read_verdict(L["v"])["ok"]
        rows.append(row)
        del L
        torch.cuda.empty_cache()
    print(json.dumps({"layer_table": args.workload, "tf32_peak_tflops": tf32_peak, "hbm_gbs": peaks["hbm_gbs"],
                      "fp32_alu_peak_tflops": FP32_ALU_PEAK_TFLOPS, "peak_source": peaks["source"],
                      "options": options, "rows": rows}), flush=True)


P_FIELD, L_FIELD = 2 ** 25 - 39, 8     # the prime and the fractional bits the paper uses (Section 5)
# Peaks of the integer tensor pipes in int8 operations (2 per multiply-accumulate) per clock and SM, as ncu states
# them for this part (sm__ops_path_tensor_op_{imma,utcimma}_src_int8_sparsity_off peak_sustained): the mma.sync
# path the field kernels use, and the tcgen05 path.  One exact multiply-accumulate of two residues costs
# sixteen u8 x u8 multiply-accumulates (four base-256 digits each).
SMS, IMMA_OPS_PER_CLK_SM, UTCIMMA_OPS_PER_CLK_SM, INT8_OPS_PER_FIELD_MAC = 148, 4096, 16384, 32


def run_field_table(args):
    """Per-layer timing of the finite-field calls (dk_field_masked_linear, dk_field_linear_bwd_wgrad) and of
    the standalone field encode / decode_verify, in exact modular multiply-accumulates per second against the
    peak of the integer tensor path each kernel runs on; a reporting aid like --layer-table."""
    import torch
    from paper_2207_00083_b200 import binding as dk
    from paper_2207_00083_b200 import synth
    dev = torch.device("cuda:0")
    torch.cuda.set_device(0)
    ctx = dk.Context(0)
    flush = torch.empty(L2_FLUSH_BYTES // 4, dtype=torch.float32, device=dev)
    out = measure_field(torch, dk, synth, ctx, dev, read_peaks(), flush, args.workload,
                        set(args.layers.split(",")) if args.layers else None, args.iters)
    print(json.dumps(out), flush=True)


def measure_field(torch, dk, synth, ctx, dev, peaks, flush, workload, want, iters):
    gen = torch.Generator(device=dev)
    gen.manual_seed(220700083)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    rows = []

    def residues(shape):
        return torch.randint(0, P_FIELD, shape, dtype=torch.int32, device=dev, generator=gen)

    def timeit(fn, iters):
        for _ in range(2):
            fn()
        tot = 0.0
        for _ in range(iters):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record()
            torch.cuda.synchronize()
            tot += a.elapsed_time(b)
        return tot / iters

    for s in synth.layers(workload):
        if want and s.name not in want:
            continue
        p = dk.problem_from_spec(s)
        ctx.ensure_workspace(p, field=True)
        rng = synth._rng(s, "coef", 7)
        C = rng.integers(1, P_FIELD, size=(s.G, s.K + 2, s.K + 1)).astype(np.uint32)
        gamma = rng.integers(1, P_FIELD, size=(s.G, s.K + 1)).astype(np.uint32)
        x = torch.empty(shape_acts(s.batch, s, "in"), device=dev)
        x.uniform_(0, 1, generator=gen) if s.x_dist == "uniform" else x.normal_(0, 1, generator=gen)
        W = torch.randn(shape_w(s), device=dev, generator=gen) * (s.w_std or (2.0 / s.kc) ** 0.5)
        rq = residues(shape_acts(s.G, s, "in"))
        y = torch.empty(shape_acts(s.batch, s, "out"), device=dev)
        xsave = torch.empty(shape_acts(s.G * (s.K + 2), s, "in"), dtype=torch.int32, device=dev)
        v = dk.new_verdict(dev.index or 0)

        def fwd():
            dk.dk_field_masked_linear(ctx, p, P_FIELD, L_FIELD, W, x, rq, C, None, y, None, xsave, v)
        row = {"layer": s.name, "M": s.cout, "Kc": s.kc, "N_fwd": s.G * (s.K + 2) * s.hout * s.wout}
        calls = [("fwd", fwd, s.fwd_flops() / 2, "linear_fwd")]
        if s.wgrad:
            dq = residues(shape_acts(s.batch, s, "out"))
            dWq = torch.empty(shape_w(s), dtype=torch.int32, device=dev)

            def wg():
                dk.dk_field_linear_bwd_wgrad(ctx, p, P_FIELD, dq, xsave, s.K + 2, C, gamma, dWq)
            calls.append(("wgrad", wg, s.wgrad_flops() / 2, "wgrad"))
        for name, fn, macs, kind in calls:
            fn()
            dk.dk_profile_reset(ctx)
            dk.dk_profile_enable(ctx, True)
            ms = timeit(fn, iters)
            prof = dk.dk_profile_read(ctx)
            dk.dk_profile_enable(ctx, False)
            kms = prof[kind][0] / max(prof[kind][1], 1)
            row[name] = {"call_ms": round(ms, 4), "kernel_ms": round(kms, 4),
                         "tmacs_call": round(macs / ms / 1e9, 3), "tmacs_kernel": round(macs / kms / 1e9, 3)}
        vd = dk.read_verdict(v)
        row["verdict_ok"] = vd["ok"]
        rows.append(row)
        torch.cuda.empty_cache()

    # standalone field encode / decode_verify on tensors much larger than L2 (uint32 residues: the same
    # bytes per position as the fp32 calls)
    K, G, n = 4, 32, 1 << 20
    spec = synth.LayerSpec("elementwise", "stream", "fc", n, n, K=K, G=G)
    p = dk.problem_from_spec(spec)
    C = np.random.default_rng(7).integers(1, P_FIELD, size=(G, K + 2, K + 1)).astype(np.uint32)
    xq, rq = residues((G * K, n)), residues((G, n))
    xbar = torch.empty((G * (K + 2), n), dtype=torch.int32, device=dev)
    yq = torch.empty((G * K, n), dtype=torch.int32, device=dev)
    v = dk.new_verdict(dev.index or 0)
    elem = {}
    for name, fn, bpp in (("encode", lambda: dk.dk_field_encode(ctx, p, P_FIELD, xq, rq, C, xbar), (2 * K + 3) * 4),
                          ("decode", lambda: dk.dk_field_decode_verify(ctx, p, P_FIELD, L_FIELD, xbar, C, None, yq,
                                                                       None, v), (2 * K + 2) * 4)):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(10):
            fn()
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / 10
        gbs = bpp * G * n / (ms * 1e-3) / 1e9
        elem[name] = {"gbs": round(gbs, 1), "frac_hbm": round(gbs / peaks["hbm_gbs"], 4), "ms": round(ms, 4)}
    assert dk.read_verdict(v)["ok"] == 1      # decode of encode-only data: rho = n . C . [x; r] = 0
    clocks = sampler.stop()
    mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
    peak = SMS * IMMA_OPS_PER_CLK_SM * mhz * 1e6 / INT8_OPS_PER_FIELD_MAC / 1e12
    peak_tc5 = SMS * UTCIMMA_OPS_PER_CLK_SM * mhz * 1e6 / INT8_OPS_PER_FIELD_MAC / 1e12
    spec_of = {s.name: s for s in synth.layers(workload)}
    for row in rows:
        for name in ("fwd", "wgrad"):
            if name in row:
                # the library's dispatch (channels-last): the forward contraction runs on tcgen05.mma.kind::i8 when
                # cin % 4 == 0, the weight gradient when stride 1 and cin, cout % 16 == 0; the rest on mma.sync
                sp = spec_of[row["layer"]]
                tc5 = (sp.cin % 4 == 0) if name == "fwd" else (sp.stride == 1 and sp.cin % 16 == 0 and sp.cout % 16 == 0)
                row[name]["path"] = "tcgen05 kind::i8" if tc5 else "mma.sync u8"
                row[name]["peak_tmacs"] = round(peak_tc5 if tc5 else peak, 2)
                row[name]["frac_of_peak_kernel"] = round(row[name]["tmacs_kernel"] / (peak_tc5 if tc5 else peak), 4)
    return {"field_table": workload, "prime": P_FIELD, "l": L_FIELD, "unit": "T exact modular MAC/s",
            "bound": "tensor (int8)", "peak_tmacs": round(peak_tc5, 2),
            "peak_source": f"{SMS} SMs x {UTCIMMA_OPS_PER_CLK_SM} int8 ops per clock and SM (ncu's peak for the "
                           f"tcgen05 int8 path; {IMMA_OPS_PER_CLK_SM} for mma.sync) x {mhz} MHz / "
                           f"{INT8_OPS_PER_FIELD_MAC} int8 ops per modular MAC",
            "mma_sync_peak_tmacs": round(peak, 2),
            "elementwise": elem, "clocks": clocks, "rows": rows}

def max_over_ranks(value, world, device):
    """Device-timed milliseconds of this rank -> the slowest rank's figure (every rank gets it).
    The replicas share nothing, so this and the barriers are the only communication of a multi-GPU run."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(flops_per_step, steps, world, ms_total):
    """Aggregate throughput of `world` replicas that each ran `steps` steps of `flops_per_step` masked
    flops within `ms_total` (the slowest rank's time), in TFLOP/s."""
    return world * flops_per_step * steps / (ms_total * 1e-3) / 1e12


# ---------------------------------------------------------------------------
# per-layer accounting: which roof binds, algorithmic bytes, issued flops
# ---------------------------------------------------------------------------
def wgrad_on_tensor_cores(s):
    """Mirror of the library's dispatch rule for the weight gradient (channels-last, default arithmetic,
    cin % 4 == 0, cout % 4 == 0, stride <= 4); everything else runs on the fp32 kernel."""
    return (getattr(s, "precision", "default") == "default" and s.cin % 4 == 0 and s.cout % 4 == 0
            and s.stride <= 4)


def algorithmic_bytes(s, call):
    """Bytes a call must move at least (fp32): the fused forward reads the K private inputs and the noise
    of every group and W once, writes the K decoded outputs and the K+1 encodings the backward pass needs;
    the weight gradient reads the K output gradients and those K+1 encodings, writes dW once."""
    if call == "fwd":
        return 4.0 * (s.G * (s.K + 1) * s.n_in + s.cout * s.kc + s.G * s.K * s.n_out + s.G * (s.K + 1) * s.n_in)
    return 4.0 * (s.G * s.K * s.n_out + s.G * (s.K + 1) * s.n_in + s.cout * s.kc)


def layer_roofs(s, call, peaks, tf32_peak):
    """Time floors of one call (ms) under the tensor roof (issued 3xTF32 flops, or fp32 FMAs for the
    kernels that do not use the tensor cores) and under the HBM roof (algorithmic bytes), and which binds."""
    flops = s.fwd_flops() if call == "fwd" else s.wgrad_flops()
    tensor = uses_tensor_cores(s) if call == "fwd" else wgrad_on_tensor_cores(s)
    issued = 3.0 * flops if tensor else flops
    fp64 = getattr(s, "precision", "default") == "fp64" and call == "fwd"     # the fp64 regime: fp64 units bind
    alu_peak = FP64_PEAK_TFLOPS if fp64 else FP32_ALU_PEAK_TFLOPS
    t_compute = issued / ((tf32_peak if tensor else alu_peak) * 1e12) * 1e3
    t_hbm = algorithmic_bytes(s, call) / (peaks["hbm_gbs"] * 1e9) * 1e3
    bound = ("tensor" if tensor else "alu") if t_compute >= t_hbm else "hbm"
    return {"bound": bound, "floor_ms": max(t_compute, t_hbm), "tensor_floor_ms": t_compute,
            "hbm_floor_ms": t_hbm, "issued_flops": issued, "tensor_cores": tensor}


def fwd_call(dk, ctx, L, fault=None, p=None):
    dk.dk_masked_linear(ctx, p or L["p"], L["W"], L["x"], L["r"], L["C"], None, L["y"], L["xsave"], L["v"], fault)


def wgrad_call(dk, ctx, L):
    s = L["spec"]
    dk.dk_linear_bwd_wgrad(ctx, L["p"], L["delta"], L["xsave"], s.K + 2, L["C"], L["gamma"], 1.0 / s.batch, L["dW"])


def profile_layers(torch, dk, ctx, layers, peaks, tf32_peak, flush, iters=2):
    """One call at a time with the library's own event pairs on: per layer and call the time of the whole
    call, of its GEMM kernel and of everything else it launches, against the roof that binds the layer."""
    rows = []
    for L in layers:
        s = L["spec"]
        row = {"layer": s.name, "M": s.cout, "Kc": s.kc, "N_fwd": s.G * (s.K + 2) * s.hout * s.wout}
        # the opt-in forward mode with W as one TF32 term (two products per step), where the tensor cores serve
        p_x2 = dk.problem_from_spec(s, precision=dk.DK_TF32X2_WUNSPLIT, tol=1e-4) if uses_tensor_cores(s) else None
        for call, fn, kind in (("fwd", lambda: fwd_call(dk, ctx, L), "linear_fwd"),
                               ("fwd_tf32x2w", lambda: fwd_call(dk, ctx, L, p=p_x2), "linear_fwd"),
                               ("wgrad", lambda: wgrad_call(dk, ctx, L), "wgrad")):
            if (call == "wgrad" and not s.wgrad) or (call == "fwd_tf32x2w" and p_x2 is None):
                continue
            fn()
            dk.dk_profile_reset(ctx)
            dk.dk_profile_enable(ctx, True)
            tot = 0.0
            for _ in range(iters):
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record()
                torch.cuda.synchronize()
                tot += a.elapsed_time(b)
            prof = dk.dk_profile_read(ctx)
            dk.dk_profile_enable(ctx, False)
            ms = tot / iters
            kms = prof[kind][0] / iters        # all GEMM launches of one call (a large layer's call has several)
            nlaunch = prof[kind][1] / iters
            if call == "fwd_tf32x2w":
                row[call] = {"call_ms": round(ms, 4), "kernel_ms": round(kms, 4),
                             "issued_tflops_kernel": round(2.0 * s.fwd_flops() / kms / 1e9, 2) if kms > 0 else None,
                             "masked_tflops_call": round(s.fwd_flops() / ms / 1e9, 2)}
                continue
            roof = layer_roofs(s, call, peaks, tf32_peak)
            flops = s.fwd_flops() if call == "fwd" else s.wgrad_flops()
            row[call] = {"bound": roof["bound"], "call_ms": round(ms, 4), "kernel_ms": round(kms, 4),
                         "kernel_launches": nlaunch,
                         # with several launches the pre-passes of later ranges run beside the GEMM of earlier
                         # ones on a second stream: their time is then no part of call - kernel
                         "other_kernels_ms": round(sum(v[0] for k, v in prof.items() if k != kind) / iters, 4),
                         "exposed_other_ms": round(ms - kms, 4),
                         "floor_ms": round(roof["floor_ms"], 4),
                         "frac_of_roof_call": round(roof["floor_ms"] / ms, 4),
                         "frac_of_roof_kernel": round(roof["floor_ms"] / kms, 4) if kms > 0 else None,
                         "masked_tflops_call": round(flops / ms / 1e9, 2),
                         "issued_tflops_kernel": round(roof["issued_flops"] / kms / 1e9, 2) if kms > 0 else None,
                         "algorithmic_gbs_call": round(algorithmic_bytes(s, call) / ms / 1e6, 1)}
        rows.append(row)
    return rows


# ---------------------------------------------------------------------------
# the ten-step schedule with one wrong accelerator output
# ---------------------------------------------------------------------------
def run_fault_schedule(dk, ctx, layers, steps=10, seed=2207):
    """`steps` passes of the whole path over all layers (fused forward with the integrity check, then the
    weight gradient); in ONE seeded (step, layer) the accelerator returns one wrong value (dk_fault).
    Returns the fault and what the verdicts said: every other call must be clean, the faulted call must
    flag exactly that element."""
    rng = np.random.default_rng(seed)
    f_step = int(rng.integers(0, steps))
    f_layer = int(rng.integers(0, len(layers)))
    s = layers[f_layer]["spec"]
    f_group, f_enc = int(rng.integers(0, s.G)), int(rng.integers(0, s.K + 2))
    f_index = int(rng.integers(0, s.n_out))
    fault = dk.dk_fault(f_group, f_enc, f_index, 500.0)
    clean_calls, bad_clean, flagged = 0, [], None
    for step in range(steps):
        for li, L in enumerate(layers):
            hit = step == f_step and li == f_layer
            fwd_call(dk, ctx, L, fault if hit else None)
            vd = dk.read_verdict(L["v"])
            if hit:
                flagged = vd
            elif (vd["ok"], vd["n_flagged"], vd["first_index"], vd["status"]) == (1, 0, -1, 0):
                clean_calls += 1
            else:
                bad_clean.append({"step": step, "layer": L["spec"].name, "verdict": vd})
            if L["spec"].wgrad:
                wgrad_call(dk, ctx, L)
    status = dk.dk_device_status(ctx)
    want_index = f_group * s.n_out + f_index
    ok = (not bad_clean and status == 0 and flagged is not None and
          (flagged["ok"], flagged["n_flagged"], flagged["first_index"]) == (0, 1, want_index))
    return {"steps": steps, "layers": len(layers), "calls_checked": steps * len(layers),
            "fault": {"step": f_step, "layer": s.name, "group": f_group, "enc": f_enc, "out_index": f_index,
                      "delta": 500.0, "expected_first_index": want_index},
            "clean_calls": clean_calls, "unexpected": bad_clean, "faulted_verdict": flagged,
            "device_status": status, "as_expected": bool(ok)}


# ---------------------------------------------------------------------------
# detection floor of the floating-point integrity check, measured through the C-ABI
# ---------------------------------------------------------------------------
def detection_floor(torch, dk, ctx, L, positions=3, iters=26):
    """Smallest wrong value that the check flags, per encoding row, found by bisection on dk_fault.delta
    (each probe is one dk_masked_linear call) at a few output elements of one layer, in units of the rms of
    that encoded output row (taken from dk_encode + dk_linear_fwd).  The paper's exact comparison has no
    such floor; the floating-point rule flags |rho| > tau * max(s_e, s_g)."""
    s, p = L["spec"], L["p"]
    E = s.K + 2
    dev = L["x"].device
    xbar = torch.empty(shape_acts(s.G * E, s, "in"), device=dev)
    ybar = torch.empty(shape_acts(s.G * E, s, "out"), device=dev)
    dk.dk_encode(ctx, p, L["x"], L["r"], L["C"], xbar)
    dk.dk_linear_fwd(ctx, p, L["W"], xbar, ybar)
    rows_rms = ybar.reshape(s.G * E, -1).square().mean(dim=1).sqrt().cpu().numpy()
    rng = np.random.default_rng(83)
    out = []
    for enc in range(E):
        floors = []
        for _ in range(positions):
            g, idx = int(rng.integers(0, s.G)), int(rng.integers(0, s.n_out))
            rms = float(rows_rms[g * E + enc])
            lo, hi = 1e-9 * rms, 1e2 * rms           # lo passes, hi is flagged
            for _ in range(iters):
                mid = (lo * hi) ** 0.5
                dk.dk_masked_linear(ctx, p, L["W"], L["x"], L["r"], L["C"], None, L["y"], None, L["v"],
                                    dk.dk_fault(g, enc, idx, mid))
                if dk.read_verdict(L["v"])["n_flagged"] >= 1:
                    hi = mid
                else:
                    lo = mid
            floors.append(hi / rms)
        out.append({"enc": enc, "floor_over_row_rms_median": float(np.median(floors)),
                    "floor_over_row_rms_max": float(max(floors))})
    dk.dk_masked_linear(ctx, p, L["W"], L["x"], L["r"], L["C"], None, L["y"], L["xsave"], L["v"])
    return {"layer": s.name, "tau": 1e-4, "rule": "flagged iff not(|rho| <= tau*max(s_e, s_g))",
            "positions_per_row": positions, "unit": "smallest flagged |delta| / rms(y_bar row)", "rows": out}


# ---------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2207_00083_b200 import binding as dk
    from paper_2207_00083_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")
    peaks = read_peaks()

    specs = synth.layers(args.workload)
    ctx = dk.Context(local)
    options = apply_options(dk, ctx, args)
    gen = torch.Generator(device=dev)
    gen.manual_seed(220700083 + rank)
    layers = [make_layer(torch, dk, synth, ctx, s, dev, gen, rank, pinned=False) for s in specs]
    biggest = max(layers, key=lambda L: ctx.workspace_bytes(L["p"]))
    ctx.ensure_workspace(biggest["p"])
    flush = torch.empty(L2_FLUSH_BYTES // 4, dtype=torch.float32, device=dev)

    def step_device():
        for L in layers:
            fwd_call(dk, ctx, L)
            if L["spec"].wgrad:
                wgrad_call(dk, ctx, L)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            flush.zero_()
            fn()
        barrier()
        evs = []
        for _ in range(steps):
            flush.zero_()                 # evict the previous step's tensors from L2 (untimed)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            evs.append((a, b))
        barrier()
        total = sum(a.elapsed_time(b) for a, b in evs)
        return max_over_ranks(total, world, dev)

    steps, warmup = max(1, args.steps), max(3, args.warmup)
    fwd_flops = sum(s.fwd_flops() for s in specs)
    wg_flops = sum(s.wgrad_flops() for s in specs if s.wgrad)
    step_flops = fwd_flops + wg_flops

    # ---- device-resident timing (the library only counts its launches here)
    for _ in range(warmup):
        flush.zero_()
        step_device()
    torch.cuda.synchronize()
    dk.dk_profile_reset(ctx)
    dk.dk_profile_enable(ctx, False)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms_total = timed(step_device, steps, 0)
    clocks = sampler.stop() if rank == 0 else None
    launches = sum(v[2] for v in dk.dk_profile_read(ctx).values())
    assert dk.dk_device_status(ctx) == 0

    # ---- a second pass with the library's per-kernel events on (the event pairs cost a little, so the step
    # metric above is taken without them): kernel shares and the dominant kernel's average launch duration,
    # measured inside the same back-to-back step
    dk.dk_profile_reset(ctx)
    dk.dk_profile_enable(ctx, True)
    prof_steps = min(steps, 10)
    timed(step_device, prof_steps, 0)
    prof = dk.dk_profile_read(ctx)
    dk.dk_profile_enable(ctx, False)

    for L in layers:        # every verdict of the last step must be clean
        vd = dk.read_verdict(L["v"])
        assert vd["ok"] == 1 and vd["status"] == 0, (L["spec"].name, vd)

    # ---- end to end through host buffers: pinned host copies of every layer's inputs and results
    e2e = measure_e2e(torch, dk, ctx, layers, dev, timed, min(steps, args.e2e_steps), step_flops, world)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    value = whole_job_value(step_flops, steps, world, ms_total)
    K = specs[0].K
    ksum = max(sum(v[0] for v in prof.values()), 1e-9)
    kernel_ms = {k: round(v[0] / max(v[1], 1), 5) for k, v in prof.items() if v[1]}
    share = {k: round(v[0] / ksum, 4) for k, v in prof.items() if v[1]}

    # roofline of the dominant kernel class (forward GEMM or wgrad GEMM), timed inside the long step: the
    # sustained tensor figure is the denominator, the burst one is given beside it
    long_step = ms_total / steps * (warmup + steps) > 1000.0
    bf16 = peaks["bf16_tflops_sustained"] if long_step else peaks["bf16_tflops"]
    tf32_peak = bf16 * TF32_OVER_BF16
    tf32_burst = peaks["bf16_tflops"] * TF32_OVER_BF16
    dom = "linear_fwd" if prof["linear_fwd"][0] >= prof["wgrad"][0] else "wgrad"
    call = "fwd" if dom == "linear_fwd" else "wgrad"
    dom_specs = [s for s in specs if call == "fwd" or s.wgrad]
    roofs = [layer_roofs(s, call, peaks, tf32_peak) for s in dom_specs]
    # a large layer's call is served by several launches (ranges of virtual batches), so the unit of this
    # object is the average launch: one step's flops and bytes over one step's launches of the class
    launches_per_step = prof[dom][1] / prof_steps
    issued_per_launch = sum(r["issued_flops"] for r in roofs) / launches_per_step
    avg_ms = prof[dom][0] / max(prof[dom][1], 1)
    achieved = issued_per_launch / (avg_ms * 1e-3) / 1e12
    alg_bytes = sum(algorithmic_bytes(s, call) for s in dom_specs) / launches_per_step
    traffic = NCU_TRAFFIC_BYTES_PER_STEP.get(args.workload, {}).get(dom)
    if traffic is not None:
        traffic = traffic / launches_per_step
    roofline = {"bound": "tensor", "achieved": achieved, "peak": tf32_peak, "unit": "TFLOP/s",
                "frac": achieved / tf32_peak, "frac_of_burst_peak": achieved / tf32_burst,
                "traffic": traffic, "traffic_unit": "bytes per launch (ncu, dram read + write, average over "
                "the step's launches of this class)", "algorithmic_bytes": alg_bytes,
                "launches_per_step": launches_per_step,
                "algorithmic_bytes_rule": "one step's calls over its launches, fp32: fused forward reads (K+1) inputs per group and W, "
                "writes K outputs and K+1 stored encodings; wgrad reads K gradients and K+1 encodings, writes dW",
                "kernel": dom, "launches_timed": prof[dom][1], "avg_launch_ms": avg_ms,
                "flops_per_launch": issued_per_launch,
                "flops": "issued flops per launch = 3 x masked flops on the tensor-core kernels (3xTF32 split), "
                         "1 x on the fp32 kernels, one step's total over one step's launches of the class",
                "peak_source": f"{peaks['source']} bf16 {'sustained' if long_step else 'burst'} {bf16} TFLOP/s "
                               f"x nominal TF32:BF16 ratio {TF32_OVER_BF16:.4f} (kernel timed inside a "
                               f"{'long' if long_step else 'short'} step)"}

    layer_rows = profile_layers(torch, dk, ctx, layers, peaks, tf32_burst, flush)
    big = [r for r in layer_rows if r["fwd"]["bound"] == "tensor"]
    elem = measure_elementwise(torch, dk, synth, ctx, dev, peaks)
    schedule = run_fault_schedule(dk, ctx, layers, steps=10)
    floor_layer = next((L for L in layers if L["spec"].name in ("fc7", "conv5_3", "layer4_3x3", "fc")), layers[-1])
    floor = detection_floor(torch, dk, ctx, floor_layer)

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_total / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "tf32x3 (fp32 in/out)", "data": "synthetic",
        "config": {"workload": args.workload, "layers": len(specs), "batch": specs[0].batch, "K": K,
                   "G": specs[0].G, "flops": "masked (all K+2 fwd / K+1 wgrad encodings)",
                   "l2": f"flushed between steps ({L2_FLUSH_BYTES >> 20} MiB write, untimed); every large "
                         f"layer's tensors exceed L2 by themselves",
                   "parallelism": "replicas only" if world > 1 else "single GPU", "options": options},
        "decoded_useful_tflops": value * (K / (K + 2) * fwd_flops + K / (K + 1) * wg_flops) / step_flops,
        "encode_gbs": elem["encode"]["gbs"], "decode_gbs": elem["decode"]["gbs"],
        "encode_frac_hbm": elem["encode"]["frac_hbm"], "decode_frac_hbm": elem["decode"]["frac_hbm"],
        "elementwise": elem,
        "kernel_ms_per_launch": kernel_ms, "kernel_time_share": share,
        "roofline": roofline,
        "layers": layer_rows,
        "layers_note": "one call at a time, L2 flushed before each, roofs from the burst tensor figure "
                       f"({tf32_burst:.1f} TFLOP/s TF32) and the measured copy bandwidth; 'bound' = the larger "
                       "of the two time floors of the call",
        "tensor_bound_layers_min_frac_kernel": min((r["fwd"]["frac_of_roof_kernel"] for r in big), default=None),
        "e2e": e2e,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "fault_schedule": schedule,
        "verify": {"detection_floor": floor},
    }
    if world == 1 and not args.no_field:
        # the finite-field calls on one mid-sized layer (reported beside the metric, measured after it;
        # `--field-table` gives every layer of a workload)
        fm = measure_field(torch, dk, synth, ctx, dev, peaks, flush, "vgg16_cifar", {"conv3_2"}, 5)
        line["field_path"] = {k: fm[k] for k in ("field_table", "prime", "l", "unit", "bound", "peak_tmacs",
                                                  "peak_source", "mma_sync_peak_tmacs", "elementwise", "rows")}
    if not args.no_cpu_baseline and world == 1:
        del layers
        torch.cuda.empty_cache()
        r = time_oracle(args.workload, len(specs), 0, budget_s=20.0)
        line["cpu_baseline"] = {"value": r["value"], "unit": "TFLOP/s", "cores": r["cores"], "kind": "oracle",
                                "sample": r["sample"]}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def measure_e2e(torch, dk, ctx, layers, dev, timed, steps, step_flops, world):
    """The same step through host buffers: every layer's inputs come from pinned host memory and its
    results go back there.  Uploads, the library's calls and downloads run on three streams chained by
    events, layer by layer, so that the copies of one layer overlap the kernels of its neighbours; a step
    starts after everything before it and ends when the last download has landed."""
    h2d = d2h = 0
    for L in layers:
        s = L["spec"]
        L["hx"] = torch.empty(L["x"].shape, dtype=torch.float32, pin_memory=True).copy_(L["x"])
        L["hr"] = torch.empty(L["r"].shape, dtype=torch.float32, pin_memory=True).copy_(L["r"])
        L["hy"] = torch.empty(L["y"].shape, dtype=torch.float32, pin_memory=True)
        L["hv"] = torch.empty(dk.VERDICT_BYTES, dtype=torch.uint8, pin_memory=True)
        h2d += (L["x"].numel() + L["r"].numel()) * 4
        d2h += L["y"].numel() * 4 + dk.VERDICT_BYTES
        if s.wgrad:
            L["hdelta"] = torch.empty(L["delta"].shape, dtype=torch.float32, pin_memory=True).copy_(L["delta"])
            L["hdW"] = torch.empty(L["W"].shape, dtype=torch.float32, pin_memory=True)
            h2d += L["delta"].numel() * 4
            d2h += L["W"].numel() * 4
    h2d_stream, d2h_stream = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    def step_e2e():
        main = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(main)
        h2d_stream.wait_event(start)
        d2h_stream.wait_event(start)
        for L in layers:
            s = L["spec"]
            with torch.cuda.stream(h2d_stream):
                L["x"].copy_(L["hx"], non_blocking=True)
                L["r"].copy_(L["hr"], non_blocking=True)
                if s.wgrad:
                    L["delta"].copy_(L["hdelta"], non_blocking=True)
                up = torch.cuda.Event()
                up.record(h2d_stream)
            main.wait_event(up)
            fwd_call(dk, ctx, L)
            fwd_done = torch.cuda.Event()
            fwd_done.record(main)
            d2h_stream.wait_event(fwd_done)
            with torch.cuda.stream(d2h_stream):
                L["hy"].copy_(L["y"], non_blocking=True)
                L["hv"].copy_(L["v"], non_blocking=True)
            if s.wgrad:
                wgrad_call(dk, ctx, L)
                wg_done = torch.cuda.Event()
                wg_done.record(main)
                d2h_stream.wait_event(wg_done)
                with torch.cuda.stream(d2h_stream):
                    L["hdW"].copy_(L["dW"], non_blocking=True)
        down = torch.cuda.Event()
        down.record(d2h_stream)
        main.wait_event(down)

    steps = max(1, steps)
    ms = timed(step_e2e, steps, 1)
    for L in layers:
        for k in ("hx", "hr", "hy", "hv", "hdelta", "hdW"):
            L.pop(k, None)
    return {"value": whole_job_value(step_flops, steps, world, ms), "unit": "TFLOP/s",
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms / steps, "steps": steps}


def run_schedule(args):
    """`--schedule`: only the ten-step schedule with one injected fault, as one JSON line."""
    import torch
    from paper_2207_00083_b200 import binding as dk
    from paper_2207_00083_b200 import synth
    dev = torch.device("cuda:0")
    torch.cuda.set_device(0)
    ctx = dk.Context(0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(220700083)
    layers = [make_layer(torch, dk, synth, ctx, s, dev, gen, 0, pinned=False) for s in synth.layers(args.workload)]
    ctx.ensure_workspace(max(layers, key=lambda L: ctx.workspace_bytes(L["p"]))["p"])
    out = run_fault_schedule(dk, ctx, layers, steps=10)
    out["workload"] = args.workload
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vgg16_224")
    ap.add_argument("--e2e-steps", type=int, default=3, help="timed steps of the host-buffer measurement")
    ap.add_argument("--no-field", action="store_true")
    ap.add_argument("--schedule", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layer-table", action="store_true")
    ap.add_argument("--field-table", action="store_true")
    ap.add_argument("--layers", default="")
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--groups", type=int, default=0,
                    help="--layer-table only: this many virtual batches per layer instead of the workload's")
    ap.add_argument("--option", action="append", default=[], metavar="NAME=VALUE",
                    help="a library option for this run, e.g. TC_CHUNK=4 (dk_set_option with DK_OPT_<NAME>); "
                         "the line then carries it under config.options")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.layer_table:
        run_layer_table(args)
    elif args.field_table:
        run_field_table(args)
    elif args.schedule:
        run_schedule(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
