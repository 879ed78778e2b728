"""The full masked VGG-16 training step at 224 x 224, batch 256 (13 convolutions
and 3 fully connected layers, K = 4, 64 virtual batches), run as the schedule
the method is meant for: ten steps of fused forward + integrity check + weight
gradient over all layers, with ONE wrong accelerator output injected in one
seeded (step, layer, group, encoding, element).  Section 4.4 and the threat
model of Section 3 fix what must come out: every honest call verifies clean,
and the tampered call flags exactly one element, the tampered one (the residual
changes by n[enc] * delta there and nowhere else).

Inputs are seeded device-side draws with the workload's shapes and
distributions; no value is compared here, only the verdicts (the decoded
values of every layer are checked against the oracle in test_gpu_fullsize.py)."""
import pytest
import torch

import bench
from paper_2207_00083_b200 import binding as dk
from paper_2207_00083_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("workload,seed", [("vgg16_224", 2207), ("vgg16_cifar", 83)])
def test_ten_steps_with_one_injected_fault(workload, seed):
    dev = torch.device("cuda:0")
    ctx = dk.Context(0)
    try:
        gen = torch.Generator(device=dev)
        gen.manual_seed(220700083)
        layers = [bench.make_layer(torch, dk, synth, ctx, s, dev, gen, 0, pinned=False) for s in synth.layers(workload)]
        ctx.ensure_workspace(max(layers, key=lambda L: ctx.workspace_bytes(L["p"]))["p"])
        out = bench.run_fault_schedule(dk, ctx, layers, steps=10, seed=seed)
        assert out["unexpected"] == []
        assert out["clean_calls"] == 10 * len(layers) - 1
        fv, f = out["faulted_verdict"], out["fault"]
        assert (fv["ok"], fv["n_flagged"], fv["first_index"], fv["status"]) == (0, 1, f["expected_first_index"], 0)
        assert out["device_status"] == 0 and out["as_expected"]
    finally:
        del layers
        ctx.close()
        torch.cuda.empty_cache()
