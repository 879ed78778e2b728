#!/usr/bin/env python
"""Benchmark of the masked linear-algebra path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload vgg16_cifar] [--no-cpu-baseline]

One step = one pass of the whole path over one synthetic batch of the
workload: for every layer the fused masked forward (encode, dense op on the
K+2 encodings, decode, integrity check, with the encodings stored) followed by
the masked weight gradient where the workload trains.  Prints ONE JSON line.

`--impl reference` times the fp64 CPU oracle as it stands on a bounded sample
of the same workload (one virtual batch of every layer per step).

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
def oracle_sample_step(specs, drawn):
    """Runs the oracle's masked forward (+ wgrad) on one group of every layer.
    Returns the masked flops it covered."""
    from oracle import dk_oracle as O
    flops = 0.0
    for spec, d in zip(specs, drawn):
        m = O.masked_forward(d["W"], d["x"], d["r"], d["C"], spec.stride, spec.pad)
        flops += spec.fwd_flops()
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
    from paper_2207_00083_b200 import synth
    specs = [s.with_groups(1) for s in synth.layers(workload)]
    drawn = [synth.draw_layer(s) for s in specs]
    for _ in range(warmup):
        oracle_sample_step(specs, drawn)
    t0 = time.perf_counter()
    flops = 0.0
    done = 0
    for _ in range(steps):
        flops += oracle_sample_step(specs, drawn)
        done += 1
        if budget_s is not None and time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    return {"value": flops / dt / 1e12, "ms_per_step": dt / done * 1e3, "steps": done,
            "sample": f"one virtual batch (G=1) of each of the {len(specs)} layers of {workload} per step, "
                      f"masked forward+verify" + (" and masked wgrad" if specs[0].wgrad else ""),
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
# our arm
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
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
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
    E = specs[0].K + 2
    gen = torch.Generator(device=dev)
    gen.manual_seed(2207_00083 + rank)

    def shape_acts(n, s, which):
        c, h, w = (s.cin, s.h, s.w) if which == "in" else (s.cout, s.hout, s.wout)
        return (n, c) if s.kind == "fc" else (n, h, w, c)

    def shape_w(s):
        return (s.cout, s.cin) if s.kind == "fc" else (s.cout, s.kh, s.kw, s.cin)

    layers = []
    h2d = d2h = 0
    for s in specs:
        p = dk.problem_from_spec(s, tol=1e-4)
        ctx.ensure_workspace(p)
        rng = synth._rng(s, "coef", rank)
        L = {"spec": s, "p": p,
             "C": synth.draw_coefficients(rng, s.K, s.G), "gamma": synth.draw_gamma(rng, s.K, s.G)}
        # pinned host copies (the end-to-end leg streams them in every step)
        hx = torch.empty(shape_acts(s.batch, s, "in"), dtype=torch.float32).pin_memory()
        hr = torch.empty(shape_acts(s.G, s, "in"), dtype=torch.float32).pin_memory()
        cpu_gen = torch.Generator().manual_seed(1000 * rank + len(layers))
        if s.x_dist == "uniform":
            hx.uniform_(0, 1, generator=cpu_gen)
        else:
            hx.normal_(0, 1, generator=cpu_gen)
        hr.normal_(0, s.sigma_r, generator=cpu_gen)
        L["hx"], L["hr"] = hx, hr
        L["x"], L["r"] = hx.to(dev), hr.to(dev)
        std = s.w_std if s.w_std is not None else (2.0 / s.kc) ** 0.5
        L["W"] = torch.randn(shape_w(s), device=dev, generator=gen) * std
        L["y"] = torch.empty(shape_acts(s.batch, s, "out"), device=dev)
        L["xsave"] = torch.empty(shape_acts(s.G * (s.K + 2), s, "in"), device=dev)
        L["v"] = dk.new_verdict(local)
        L["hy"] = torch.empty(shape_acts(s.batch, s, "out"), dtype=torch.float32).pin_memory()
        L["hv"] = torch.empty(dk.VERDICT_BYTES, dtype=torch.uint8).pin_memory()
        h2d += hx.numel() * 4 + hr.numel() * 4
        d2h += L["hy"].numel() * 4 + dk.VERDICT_BYTES
        if s.wgrad:
            hd = torch.empty(shape_acts(s.batch, s, "out"), dtype=torch.float32).pin_memory()
            hd.normal_(0, 1, generator=cpu_gen)
            L["hdelta"], L["delta"] = hd, hd.to(dev)
            L["dW"] = torch.empty_like(L["W"])
            L["hdW"] = torch.empty(shape_w(s), dtype=torch.float32).pin_memory()
            h2d += hd.numel() * 4
            d2h += L["hdW"].numel() * 4
        layers.append(L)
    # the workspace may have been re-allocated while growing: register the final one per layer
    biggest = max(layers, key=lambda L: ctx.workspace_bytes(L["p"]))
    ctx.ensure_workspace(biggest["p"])

    flush = torch.empty(L2_FLUSH_BYTES // 4, dtype=torch.float32, device=dev)

    def step_device():
        for L in layers:
            s = L["spec"]
            dk.dk_masked_linear(ctx, L["p"], L["W"], L["x"], L["r"], L["C"], None, L["y"], L["xsave"], L["v"])
            if s.wgrad:
                dk.dk_linear_bwd_wgrad(ctx, L["p"], L["delta"], L["xsave"], s.K + 2, L["C"], L["gamma"],
                                       1.0 / s.batch, L["dW"])

    def step_e2e():
        for L in layers:
            s = L["spec"]
            L["x"].copy_(L["hx"], non_blocking=True)
            L["r"].copy_(L["hr"], non_blocking=True)
            dk.dk_masked_linear(ctx, L["p"], L["W"], L["x"], L["r"], L["C"], None, L["y"], L["xsave"], L["v"])
            L["hy"].copy_(L["y"], non_blocking=True)
            L["hv"].copy_(L["v"], non_blocking=True)
            if s.wgrad:
                L["delta"].copy_(L["hdelta"], non_blocking=True)
                dk.dk_linear_bwd_wgrad(ctx, L["p"], L["delta"], L["xsave"], s.K + 2, L["C"], L["gamma"],
                                       1.0 / s.batch, L["dW"])
                L["hdW"].copy_(L["dW"], non_blocking=True)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            flush.zero_()
            fn()
        barrier()
        total = 0.0
        evs = []
        for _ in range(steps):
            flush.zero_()                 # evict the previous step's tensors from L2 (untimed)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            evs.append((a, b))
        barrier()
        for a, b in evs:
            total += a.elapsed_time(b)
        t = torch.tensor([total], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    steps, warmup = max(1, args.steps), max(3, args.warmup)
    fwd_flops = sum(s.fwd_flops() for s in specs)
    wg_flops = sum(s.wgrad_flops() for s in specs if s.wgrad)
    step_flops = fwd_flops + wg_flops

    # ---- device-resident timing, with per-kernel events inside the library
    for _ in range(warmup):
        step_device()
    torch.cuda.synchronize()
    dk.dk_profile_reset(ctx)
    dk.dk_profile_enable(ctx, True)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms_total = timed(step_device, steps, 0)
    clocks = sampler.stop() if rank == 0 else None
    prof = dk.dk_profile_read(ctx)
    dk.dk_profile_enable(ctx, False)
    launches = sum(v[2] for v in prof.values())

    # ---- end to end through host buffers
    ms_e2e = timed(step_e2e, steps, 1)

    # every verdict of the last step must be clean
    for L in layers:
        vd = dk.read_verdict(L["v"])
        assert vd["ok"] == 1 and vd["status"] == 0, (L["spec"].name, vd)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    value = world * step_flops * steps / (ms_total * 1e-3) / 1e12
    e2e_value = world * step_flops * steps / (ms_e2e * 1e-3) / 1e12
    K = specs[0].K

    # roofline of the dominant kernel class
    dom = max(prof, key=lambda k: prof[k][0])
    kernel_ms = {k: round(v[0] / max(v[1], 1), 5) for k, v in prof.items() if v[1]}
    share = {k: round(v[0] / max(sum(x[0] for x in prof.values()), 1e-9), 4) for k, v in prof.items() if v[1]}
    issued_per_flop = 1.0   # SIMT fp32: one FMA per multiply-add
    if dom in ("linear_fwd", "wgrad"):
        flops_launch = (fwd_flops if dom == "linear_fwd" else wg_flops) / len(
            [s for s in specs if (dom == "linear_fwd" or s.wgrad)])
        avg_ms = prof[dom][0] / max(prof[dom][1], 1)
        achieved = flops_launch * issued_per_flop / (avg_ms * 1e-3) / 1e12
        peak = 148 * 128 * 2 * (clocks["sm_max_mhz"] or 1965.0) * 1e6 / 1e12
        roofline = {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                    "frac": achieved / peak, "traffic": None, "kernel": dom,
                    "peak_source": "148 SMs x 128 fp32 FMA lanes x 2 flop x max SM clock (derived)"}
    else:
        per_pos = {"encode": (K + 1 + K + 2) * 4, "decode_verify": (K + 2 + K) * 4, "mix_delta": (2 * K + 1) * 4}
        nel = {"encode": sum(s.G * s.n_in for s in specs), "decode_verify": sum(s.G * s.n_out for s in specs),
               "mix_delta": sum(s.G * s.n_out for s in specs if s.wgrad)}.get(dom, 0)
        nl = len(specs)
        avg_ms = prof[dom][0] / max(prof[dom][1], 1)
        achieved = per_pos.get(dom, 0) * nel / nl / (avg_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "traffic": None, "kernel": dom,
                    "peak_source": peaks["source"]}

    def gbs(kind, bytes_per_pos, nel):
        if kind not in prof or not prof[kind][1]:
            return None
        per_step_ms = prof[kind][0] / steps
        return bytes_per_pos * nel / (per_step_ms * 1e-3) / 1e9

    enc_gbs = gbs("encode", (2 * K + 3) * 4, sum(s.G * s.n_in for s in specs))
    dec_gbs = gbs("decode_verify", (2 * K + 2) * 4, sum(s.G * s.n_out for s in specs))

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_total / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "layers": len(specs), "batch": specs[0].batch, "K": K,
                   "G": specs[0].G, "flops": "masked (all K+2 fwd / K+1 wgrad encodings)",
                   "l2": f"flushed between steps ({L2_FLUSH_BYTES >> 20} MiB write, untimed)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "decoded_useful_tflops": value * (K / (K + 2) * fwd_flops + K / (K + 1) * wg_flops) / step_flops,
        "encode_gbs": enc_gbs, "decode_gbs": dec_gbs,
        "encode_frac_hbm": None if enc_gbs is None else enc_gbs / peaks["hbm_gbs"],
        "decode_frac_hbm": None if dec_gbs is None else dec_gbs / peaks["hbm_gbs"],
        "kernel_ms_per_launch": kernel_ms, "kernel_time_share": share,
        "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e / steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if not args.no_cpu_baseline and world == 1:
        r = time_oracle(args.workload, 500, 1, budget_s=12.0)
        line["cpu_baseline"] = {"value": r["value"], "unit": "TFLOP/s", "cores": r["cores"], "kind": "oracle",
                                "sample": r["sample"]}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vgg16_cifar")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
