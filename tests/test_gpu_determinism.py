"""Run-to-run reproducibility: no kernel of the layer sums in an order that depends on scheduling (no floating-point
atomics; the dynamically scheduled weight-gradient kernel hands out work items at run time but every output element
is produced by one item, and the parts of a split expert are added in a fixed order), so two runs on the same inputs
must agree bit for bit, whatever ran on the GPU in between."""
import pytest

from paper_2502_16927_b200 import workloads as wl

from helpers import empty_grads, make_layer, to_device
from test_gpu_parity import conditioned

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("case", [
    dict(shape=dict(T=6000, d=256, r=256, h=512, E=16, k=2), flags=wl.FLAG_DYNAMIC_WGRAD, kw=dict()),
    dict(shape=dict(T=5000, d=256, r=128, h=256, E=24, k=3), flags=0, kw=dict(capacity_factor=1.0, aux_loss_coef=5.0)),
    dict(shape=dict(T=3000, d=128, r=64, h=128, E=8, k=2), flags=0, kw=dict(), bias=True),
])
def test_two_runs_agree_bit_for_bit(case):
    import numpy as np
    import torch

    w = wl.Workload("det", dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=131, expert_bias=case.get("bias", False), **case["shape"])
    inp = conditioned(w)
    inp["b_gate"] = (3.0 * np.linspace(1.0, -1.0, w.E) ** 3).astype(np.float32)       # long and short segments
    dev = to_device(w, inp)
    runs = []
    for attempt in range(2):
        layer = make_layer(w, case["flags"], **case["kw"])
        y = layer.forward(dev["x"], dev, training=True)
        G = empty_grads(w, "cuda", fill=float("nan"))
        dx = layer.backward(dev["x"], dev["dy"], dev, G)
        torch.cuda.synchronize()
        assert layer.status() == 0
        runs.append(dict(G, y=y.clone(), dx=dx.clone()))
        layer.close()
        if attempt == 0:                                   # disturb the GPU's state between the runs
            junk = torch.randn(4096, 4096, device="cuda")
            (junk @ junk).sum().item()
    for key, val in runs[0].items():
        assert torch.equal(val.view(torch.uint8), runs[1][key].view(torch.uint8)), key
