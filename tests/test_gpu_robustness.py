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


def test_a_wait_that_runs_out_is_reported_and_leaves_the_handle_usable():
    """Failure path of the device-side waits, made without a fault: a one-thread kernel polls, with the pipelines'
    bounded wait and a short limit, a barrier nobody arrives at; it gives up, records that in the status word and
    returns.  The host reads BIGMAC_ERR_TIMEOUT once; the same handle then computes a correct step."""
    import numpy as np
    import torch

    import oracle
    from paper_2502_16927_b200 import binding
    from helpers import to_numpy

    w = wl.Workload("to", T=300, d=128, r=64, h=128, E=8, k=2, dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=139)
    inp = conditioned(w)
    dev = to_device(w, inp)
    layer = make_layer(w)
    assert layer.status() == 0
    binding.bigmac_debug_expire_wait(layer.handle)
    assert layer.status() == -5                            # BIGMAC_ERR_TIMEOUT
    assert layer.status() == 0                             # cleared by the read
    y = layer.forward(dev["x"], dev, training=False)
    torch.cuda.synchronize()
    assert layer.status() == 0
    ref = oracle.forward_tokens(inp, oracle.route(inp, w.k), w.act)["y"]
    assert oracle.max_rel_err(to_numpy(y), ref) <= 2e-2
    layer.close()
