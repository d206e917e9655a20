"""bigmac_route_static: routing for callers that cannot allocate device memory (a host whose memory pool
owns all free HBM, a latency-critical loop that must avoid cudaMalloc's implicit synchronisation, a plug-in
that only receives input and output pointers).  Its intermediates live in a fixed device array inside the
library instead of a caller-provided scratch buffer.

The check: through the C ABI, on the same inputs, it must return exactly the tables bigmac_route returns -
twice in a row, because the array keeps the previous call's contents - it must leave the device's free memory
as it found it, and it must refuse a problem that does not fit the array.  The variants whose routing needs more
intermediates (a load-balancing loss, a gate that reads x') go through the same comparison.  Collected last on
purpose, and independent of what ran before it."""
import numpy as np
import pytest

from paper_2502_16927_b200 import workloads as wl

from helpers import make_layer, to_device

pytestmark = pytest.mark.gpu

TABLES = ("topk_idx", "topk_w", "counts", "offsets", "row_of_slot", "slot_of_row")


def _same(a, b):
    for key in TABLES:
        np.testing.assert_array_equal(a[key].cpu().numpy(), b[key].cpu().numpy(), err_msg=key)


@pytest.mark.parametrize("name,T,variant", [("tiny", 256, {}), ("small", 2048, {}), ("tiny", 200, {"aux_loss_coef": 0.01}),
                                            ("tiny", 200, {"gate_low": True})])
def test_route_static_matches_route_twice_in_a_row(name, T, variant):
    import dataclasses

    import torch
    from paper_2502_16927_b200 import binding

    w = wl.WORKLOADS[name].with_tokens(T)
    kw = {}
    if variant.get("gate_low"):
        w = dataclasses.replace(w, gate_low=True)
    if "aux_loss_coef" in variant:
        kw["aux_loss_coef"] = variant["aux_loss_coef"]
    inp = wl.make_inputs(w)
    dev = to_device(w, inp)
    layer = make_layer(w, **kw)
    expected = layer.route(dev["x"], dev)                       # existing entry point, caller-provided scratch
    torch.cuda.synchronize()
    other = to_device(w, wl.make_inputs(w.with_tokens(T, seed=w.seed + 7)))
    for call in range(2):
        got = layer.empty_routing(T)
        for t in got.values():
            t.fill_(-1)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0] if call == 1 else None
        binding.bigmac_route_static(layer.handle, dev["x"], T, dev, got)
        torch.cuda.synchronize()
        if call == 1:                                           # the set-up call is behind us: free memory does not move
            assert torch.cuda.mem_get_info()[0] == free_before
        _same(got, expected)
        if "aux_loss_coef" in variant:
            assert got["aux_loss"].item() == expected["aux_loss"].item() > 0
        if call == 0:                                           # leave different contents behind in the array
            junk = layer.empty_routing(T)
            binding.bigmac_route_static(layer.handle, other["x"], T, other, junk)
            torch.cuda.synchronize()
    assert layer.status() == 0
    layer.close()


def test_route_static_rejects_what_does_not_fit():
    import torch
    from paper_2502_16927_b200 import binding

    w = wl.Workload("big", T=32768, d=64, r=64, h=64, E=128, k=8, dtype=wl.DTYPE_BF16, act=wl.ACT_RELU, seed=3)
    layer = make_layer(w)
    x = torch.zeros(w.T, w.d, dtype=torch.bfloat16, device="cuda")
    W = {"w_gate": torch.zeros(w.E, w.d, dtype=torch.bfloat16, device="cuda"),
         "w_down": torch.zeros(w.r, w.d, dtype=torch.bfloat16, device="cuda"),
         "w1": torch.zeros(w.E, w.h, w.r, dtype=torch.bfloat16, device="cuda"),
         "w2": torch.zeros(w.E, w.r, w.h, dtype=torch.bfloat16, device="cuda"),
         "w_up": torch.zeros(w.d, w.r, dtype=torch.bfloat16, device="cuda")}
    out = layer.empty_routing(w.T)
    for t in out.values():
        t.fill_(-1)
    with pytest.raises(binding.BigmacError) as e:
        binding.bigmac_route_static(layer.handle, x, w.T, W, out)
    assert e.value.status == -7
    torch.cuda.synchronize()
    assert all(bool((t == -1).all()) for t in out.values())     # nothing was launched
    layer.close()
