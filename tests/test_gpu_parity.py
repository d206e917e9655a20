"""GPU parity: the CUDA layer, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Integer tables must match bit for bit; floats within the stated tolerances
(max-relative error with the denominator floored at the reference tensor's RMS):
1e-4 for the fp32 path, 2e-2 for the BF16 path (bf16 storage, fp32 accumulation)."""
import numpy as np
import pytest

import oracle
from oracle import margin
from paper_2502_16927_b200 import workloads as wl

from helpers import empty_grads, make_layer, to_device, to_numpy

pytestmark = pytest.mark.gpu

TOL = {wl.DTYPE_F32: 1e-4, wl.DTYPE_BF16: 2e-2}
SIMT = 1


def conditioned(w):
    inp = wl.make_inputs(w)
    margin.enforce_margin(w, inp, 1e-3)
    return inp


def check_routing(R, rt):
    np.testing.assert_array_equal(to_numpy(R["topk_idx"]).reshape(rt.topk_idx.shape), rt.topk_idx)
    np.testing.assert_array_equal(to_numpy(R["counts"]), rt.counts)
    np.testing.assert_array_equal(to_numpy(R["offsets"]), rt.offsets)
    np.testing.assert_array_equal(to_numpy(R["row_of_slot"]), rt.row_of_slot)
    np.testing.assert_array_equal(to_numpy(R["slot_of_row"]), rt.slot_of_row)
    np.testing.assert_allclose(to_numpy(R["topk_w"]).reshape(rt.topk_p.shape), rt.topk_p, rtol=0, atol=2e-5)


def run_full(w, inp, flags=0):
    """Forward (training) + backward on the GPU; returns numpy results keyed like the oracle's."""
    import torch

    dev = to_device(w, inp)
    layer = make_layer(w, flags)
    y, R = layer.forward(dev["x"], dev, training=True, want_routing=True)
    G = empty_grads(w, "cuda", fill=float("nan"))
    dx = layer.backward(dev["x"], dev["dy"], dev, G, accumulate=False)
    torch.cuda.synchronize()
    assert layer.status() == 0
    out = {"y": to_numpy(y), "dx": to_numpy(dx), "routing": R}
    out.update({key: to_numpy(val) for key, val in G.items()})
    layer.close()
    return out


def compare_full(w, inp, got, tol):
    rt = oracle.route(inp, w.k)
    check_routing(got["routing"], rt)
    ref = oracle.backward_full(inp, rt, w.act)
    errs = {"y": oracle.rel_err(got["y"], ref["y"]), "dx": oracle.rel_err(got["dx"], ref["dx"]),
            "dw_up": oracle.rel_err(got["dw_up"], ref["dw_up"]),
            "dw_down": oracle.rel_err(got["dw_down"], ref["dw_down"]),
            "dw_gate": oracle.rel_err(got["dw_gate"], ref["dw_gate"]),
            "dw1": oracle.rel_err(got["dw1"], np.stack([ref["dw1"][e] for e in range(w.E)])),
            "dw2": oracle.rel_err(got["dw2"], np.stack([ref["dw2"][e] for e in range(w.E)]))}
    if inp.get("b_gate") is not None or True:
        errs["db_gate"] = oracle.rel_err(got["db_gate"], ref["db_gate"])
    bad = {key: val for key, val in errs.items() if not val <= tol}
    assert not bad, (bad, errs)
    for e in range(w.E):                                   # experts without tokens: exactly zero gradients
        if rt.counts[e] == 0:
            assert not got["dw1"][e].any() and not got["dw2"][e].any()
    return errs


def test_tiny_fp32_forward_backward():
    w = wl.WORKLOADS["tiny"]
    inp = conditioned(w)
    compare_full(w, inp, run_full(w, inp), TOL[wl.DTYPE_F32])


@pytest.mark.parametrize("shape", [
    dict(T=1, d=16, r=8, h=12, E=8, k=3),       # single token: most experts empty
    dict(T=77, d=20, r=12, h=28, E=5, k=5),     # k = E (dense mixture), ragged sizes
    dict(T=130, d=16, r=8, h=8, E=1, k=1),      # one expert, more than one row tile
    dict(T=5, d=8, r=4, h=4, E=16, k=1),        # fewer slots than experts
    dict(T=300, d=36, r=20, h=44, E=7, k=2),    # nothing a multiple of a tile
])
@pytest.mark.parametrize("act", [wl.ACT_RELU, wl.ACT_GELU_ERF, wl.ACT_GELU_TANH])
def test_fp32_edge_shapes(shape, act):
    w = wl.Workload("edge", dtype=wl.DTYPE_F32, act=act, seed=99 + act, **shape)
    inp = conditioned(w)
    inp["b_gate"] = (np.linspace(-0.3, 0.3, w.E)).astype(np.float32)
    margin.enforce_margin(w, inp, 1e-3)
    compare_full(w, inp, run_full(w, inp), TOL[wl.DTYPE_F32])


def test_small_bf16_fma_contractions():
    """The BF16 layer with every contraction on the plain-FMA kernels (isolates everything but tcgen05)."""
    w = wl.WORKLOADS["small"].with_tokens(1024)
    inp = conditioned(w)
    compare_full(w, inp, run_full(w, inp, flags=SIMT), TOL[wl.DTYPE_BF16])


def test_route_matches_forward_tables_and_zero_tokens_is_a_noop():
    import torch

    w = wl.WORKLOADS["tiny"]
    inp = conditioned(w)
    dev = to_device(w, inp)
    layer = make_layer(w)
    R = layer.route(dev["x"], dev)
    torch.cuda.synchronize()
    check_routing(R, oracle.route(inp, w.k))
    empty = dev["x"][:0].contiguous()
    y = layer.forward(empty, dev)
    assert y.shape[0] == 0 and layer.status() == 0
    layer.close()


def test_accumulate_adds_to_existing_gradients():
    import torch

    w = wl.WORKLOADS["tiny"]
    inp = conditioned(w)
    dev = to_device(w, inp)
    layer = make_layer(w)
    layer.forward(dev["x"], dev, training=True)
    G0 = empty_grads(w, "cuda", fill=0.0)
    layer.backward(dev["x"], dev["dy"], dev, G0, accumulate=False)
    layer.forward(dev["x"], dev, training=True)
    G1 = empty_grads(w, "cuda", fill=0.5)
    layer.backward(dev["x"], dev["dy"], dev, G1, accumulate=True)
    torch.cuda.synchronize()
    for key in G0:
        np.testing.assert_allclose(to_numpy(G1[key]), to_numpy(G0[key]) + 0.5, rtol=1e-5, atol=1e-5)
    layer.close()


def test_argument_errors_launch_nothing():
    import torch
    from paper_2502_16927_b200 import binding

    w = wl.WORKLOADS["tiny"]
    inp = conditioned(w)
    dev = to_device(w, inp)
    layer = make_layer(w)
    y = torch.zeros_like(dev["x"])
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.BigmacError) as e:
        binding.bigmac_forward(layer.handle, dev["x"], w.T, dev, y, None, None, small)
    assert e.value.status == -3                                            # workspace too small
    with pytest.raises(binding.BigmacError) as e:
        binding.bigmac_forward(layer.handle, dev["x"], w.T + 1, dev, y, None, None, small)
    assert e.value.status == -1                                            # T > max_tokens
    with pytest.raises(RuntimeError):
        layer.backward(dev["x"], dev["dy"], dev, empty_grads(w, "cuda"))   # no training forward yet
    torch.cuda.synchronize()
    assert not y.any() and layer.status() == 0
    layer.close()


def test_exchange_rows_dispatch_then_unit_combine_is_k_copies():
    """Dispatch followed by the combine, on rows of width r and of width d (the fine-grained layer's
    exchange width, Eq. 1): with the gate values of a token summing to 1, identical copies of a row
    combine back to the row itself."""
    import torch

    w = wl.WORKLOADS["tiny"]
    inp = conditioned(w)
    dev = to_device(w, inp)
    layer = make_layer(w)
    layer.forward(dev["x"], dev, training=True)
    for width, src in ((w.d, dev["x"]), (w.r, dev["x"][:, : w.r].contiguous())):
        P = ((w.N + 127) // 128 + w.E) * 128
        grouped = torch.full((P, width), float("nan"), dtype=src.dtype, device="cuda")
        dst = torch.empty_like(src)
        binding_exchange(layer, w, width, src, grouped, dst)
        torch.cuda.synchronize()
        np.testing.assert_allclose(to_numpy(dst), to_numpy(src), rtol=2e-6, atol=1e-6)
    layer.close()


def binding_exchange(layer, w, width, src, grouped, dst):
    from paper_2502_16927_b200 import binding

    binding.bigmac_exchange_rows(layer.handle, layer._saved, w.T, width, src, grouped, dst, 2)
