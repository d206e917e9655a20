"""GPU parity: the CUDA layer, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Integer tables must match bit for bit.  Floats, per output tensor:
  fp32 path  max_i |a_i-b_i| / max(|b_i|, rms(b)) <= 1e-4   (every element, denominator floored at the RMS);
  BF16 path  max_i |a_i-b_i| / max_i |b_i| <= 1e-2,  ||a-b||_F / ||b||_F <= 8e-3,  and the RMS-floored metric of
             the fp32 path <= 6e-2 (per expert for the stacked per-expert gradients).
The BF16 layer stores five (forward) to eight (gradients) intermediates per output in bf16 (unit roundoff
2^-8): each storage adds noise of about 0.165 % of the tensor's RMS, so the extreme element of 10^6..10^8
outputs sits at 2-2.5 % of the RMS even with exact accumulation (test_precision_model.py shows this with an
emulation: per-element noise of 0.47 % of the RMS after eight storages, whose extreme over 10^8 elements lies near
seven standard deviations), and where the rows of a tensor differ in scale (skewed routing, dropped slots) the
storage noise of the large rows reaches elements that sit at the floor: measured up to 5.0e-2 (dx under a capacity
limit), so the RMS-floored metric is reported and bounded at 6e-2 only, and the two bounds
that do the discriminating are set at about twice what the kernels deliver: the largest error relative to the
largest magnitude (measured 0.35-0.5 %) and the Frobenius error (measured 0.35-0.6 %), so that an error of a
few per cent of the RMS in isolated elements, or a per-cent-level systematic one, fails."""
import numpy as np
import pytest

import oracle
from oracle import margin
from paper_2502_16927_b200 import workloads as wl

from helpers import oracle_inputs, empty_grads, make_layer, to_device, to_numpy

pytestmark = pytest.mark.gpu

BF16_MAX, BF16_FRO, BF16_RMS = 1e-2, 8e-3, 6e-2
# Tensors with bounds of their own (max-norm, Frobenius), measured worst values in brackets:
#   dw1, dw2   a per-expert gradient is a sum over that expert's rows only; with a handful of rows (the sampled
#              full-size checks, nearly empty experts) the storage error of the terms does not average out and the
#              largest elements carry it whole (0.92 % of max|b| at the large workload, Frobenius 0.48 %);
#   db_gate    a sum of terms of both signs that cancels to a small difference of large parts under skewed routing;
#              the bf16 storage of dy' and u behind every term is then a larger share of the result (1.6 % / 1.0 %);
#   dw_gate    its rows are dl_j x: every dl_j = p_j (dp_j - g) is itself a difference of dot products of bf16-stored
#              rows, and with a handful of tokens nothing averages that out (Frobenius 1.2 % for a single token).
#   Their RMS-floored metric (one floor per expert) is bounded at 1e-1: an element of a per-expert gradient is a sum of
#   products of two Gaussian-like factors, and where one large term dominates a small sum its storage error is several
#   per cent of the expert's RMS (measured up to 8.0e-2 on the medium workload's sampled check).
BF16_OWN = {"dw1": (1.5e-2, BF16_FRO, 1e-1), "dw2": (1.5e-2, BF16_FRO, 1e-1), "db_gate": (2e-2, 1.5e-2, BF16_RMS),
            "dw_gate": (1.5e-2, 1.5e-2, BF16_RMS)}
# ReLU' flips (see RELU_DECISION_KEYS below) are counted against twice the max-norm bound.
RELU_OUTLIER = 2 * BF16_MAX
TOL = {wl.DTYPE_F32: 1e-4, wl.DTYPE_BF16: BF16_MAX}
SIMT = 1


def conditioned(w):
    inp = wl.make_inputs(w)
    margin.enforce_margin(w, inp, 1e-3)
    return inp


def check_routing(R, rt, p_atol=2e-5):
    np.testing.assert_array_equal(to_numpy(R["topk_idx"]).reshape(rt.topk_idx.shape), rt.topk_idx)
    np.testing.assert_array_equal(to_numpy(R["counts"]), rt.counts)
    np.testing.assert_array_equal(to_numpy(R["offsets"]), rt.offsets)
    np.testing.assert_array_equal(to_numpy(R["row_of_slot"]), rt.row_of_slot)
    np.testing.assert_array_equal(to_numpy(R["slot_of_row"]), rt.slot_of_row)
    np.testing.assert_array_equal(to_numpy(R["counts_chosen"]), rt.counts_chosen)
    np.testing.assert_allclose(to_numpy(R["topk_w"]).reshape(rt.topk_p.shape), rt.topk_p, rtol=0, atol=p_atol)


def run_full(w, inp, flags=0, capacity_factor=0.0, aux=0.0):
    """Forward (training) + backward on the GPU; returns numpy results keyed like the oracle's."""
    import torch

    dev = to_device(w, inp)
    layer = make_layer(w, flags, capacity_factor=capacity_factor, aux_loss_coef=aux)
    y, R = layer.forward(dev["x"], dev, training=True, want_routing=True)
    G = empty_grads(w, "cuda", fill=float("nan"))
    dx = layer.backward(dev["x"], dev["dy"], dev, G, accumulate=False)
    torch.cuda.synchronize()
    assert layer.status() == 0
    out = {"y": to_numpy(y), "dx": to_numpy(dx), "routing": R, "aux_loss": float(R["aux_loss"].item())}
    out.update({key: to_numpy(val) for key, val in G.items()})
    layer.close()
    return out


def float_errors(w, got, ref):
    """Per output tensor: the gate metric of the workload's dtype; for BF16 also the Frobenius error (":fro") and the
    RMS-floored elementwise metric (":rms")."""
    metric = oracle.rel_err if w.dtype == wl.DTYPE_F32 else oracle.max_rel_err
    out = {}
    for key in got:
        if key in ref:
            out[key] = metric(got[key], ref[key])
            if w.dtype == wl.DTYPE_BF16:
                out[key + ":fro"] = oracle.fro_rel_err(got[key], ref[key])
                a, b = np.asarray(got[key]), np.asarray(ref[key])
                if key in ("dw1", "dw2") and b.ndim == 3:      # one RMS floor per expert: their scales differ with their loads
                    out[key + ":rms"] = max(oracle.rel_err(a[e], b[e]) for e in range(b.shape[0]))
                else:
                    out[key + ":rms"] = oracle.rel_err(a, b)
    return out


def tolerance_of(w, key):
    if w.dtype == wl.DTYPE_F32:
        return TOL[wl.DTYPE_F32]
    base, _, suffix = key.partition(":")
    own_max, own_fro, own_rms = BF16_OWN.get(base, (BF16_MAX, BF16_FRO, BF16_RMS))
    return own_fro if suffix == "fro" else own_rms if suffix == "rms" else own_max


def assert_within(w, errs):
    record_errors(w, errs)
    bad = {key: val for key, val in errs.items() if not val <= tolerance_of(w, key)}
    assert not bad, (bad, errs)


# Worst value of every metric seen per workload name during the run, written next to the test log so that the
# measured margins can be quoted (tests never read it back).
_WORST = {}


def record_errors(w, errs):
    import json
    import os

    slot = _WORST.setdefault(w.name, {})
    for key, val in errs.items():
        slot[key] = max(slot.get(key, 0.0), float(val))
    out = os.environ.get("BIGMAC_ERROR_REPORT")
    if out:
        with open(out, "w") as f:
            json.dump(_WORST, f, indent=1, sort_keys=True)


def outlier_fraction(a, b, tol):
    """Share of elements whose error exceeds tol * max|b|."""
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.mean(np.abs(a - b) > tol * np.max(np.abs(b))))


# Gradients that pass through sigma'.  With ReLU in BF16, sigma'(z) = [z > 0] is a discrete decision taken
# on z values that carry the rounding of x' (and its fp32 accumulation order): the oracle takes it from
# the bf16-rounded x' as well, but a handful of hidden units with |z| inside the accumulation noise still
# decide differently.  Each such unit changes isolated gradient elements, so for those tensors an elementwise
# bound (2e-2 of the largest magnitude) is required of all but 1e-3 of the elements and the Frobenius bound of the
# whole tensor.
RELU_DECISION_KEYS = ("dx", "dw1", "dw2", "dw_down", "dw_gate", "db_gate", "db1")


def compare_full(w, inp, got, tol=None, capacity_factor=0.0, aux=0.0):
    inp = oracle_inputs(w, inp)
    rt = oracle.route(inp, w.k, capacity_factor=capacity_factor)
    check_routing(got["routing"], rt)
    ref = oracle.backward_full(inp, rt, w.act, decide_bf16=w.dtype == wl.DTYPE_BF16, aux_alpha=aux)
    # the loss is a sum of T*E fp32 terms on the GPU: 1e-5 relative covers its rounding at every size used here
    assert abs(got["aux_loss"] - ref.get("aux_loss", 0.0)) <= 1e-5 * abs(ref.get("aux_loss", 0.0))
    ref["dw1"] = np.stack([ref["dw1"][e] for e in range(w.E)])
    ref["dw2"] = np.stack([ref["dw2"][e] for e in range(w.E)])
    keys = (("y", "dx", "dw_gate", "dw1", "dw2", "db_gate") + (() if w.cdac else ("dw_up", "dw_down")) +
            (("db1", "db2") if w.expert_bias else ()))
    errs = float_errors(w, {key: got[key] for key in keys}, ref)
    if w.dtype == wl.DTYPE_BF16 and w.act == wl.ACT_RELU:
        for key in RELU_DECISION_KEYS:
            if key not in keys:
                continue
            assert outlier_fraction(got[key], ref[key], RELU_OUTLIER) <= 1e-3, key
            errs.pop(key)
            errs.pop(key + ":rms")
    assert_within(w, errs)
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
    dict(T=33, d=16, r=8, h=8, E=48, k=40),     # more than 32 experts per token
    dict(T=700, d=16, r=8, h=8, E=1024, k=3),   # the largest expert count the library takes; most experts empty
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
    compare_full(w, inp, run_full(w, inp, flags=SIMT))


def test_small_bf16_full_config():
    """configs[1]: T=4096, d=1024, r=128, E=32, k=4, h=512, GELU, BF16, every contraction on tcgen05."""
    w = wl.WORKLOADS["small"]
    inp = conditioned(w)
    compare_full(w, inp, run_full(w, inp))


@pytest.mark.parametrize("shape", [
    dict(T=1, d=64, r=64, h=64, E=8, k=3),         # single token, most experts empty
    dict(T=77, d=128, r=64, h=192, E=5, k=5),      # k = E, E not a multiple of 8, ragged T
    dict(T=130, d=64, r=128, h=64, E=1, k=1),      # one expert
    dict(T=300, d=192, r=64, h=128, E=40, k=2),    # E between tile sizes
    dict(T=1000, d=256, r=192, h=320, E=16, k=4),  # widths that are odd multiples of 64
    dict(T=3000, d=64, r=64, h=64, E=1024, k=2),   # the largest expert count: a few rows per expert, 1024 padded tiles
])
@pytest.mark.parametrize("act", [wl.ACT_RELU, wl.ACT_GELU_ERF])
def test_bf16_edge_shapes(shape, act):
    w = wl.Workload("edge", dtype=wl.DTYPE_BF16, act=act, seed=199 + act, **shape)
    inp = conditioned(w)
    inp["b_gate"] = (np.linspace(-0.3, 0.3, w.E)).astype(np.float32)
    margin.enforce_margin(w, inp, 1e-3)
    compare_full(w, inp, run_full(w, inp))


def test_bf16_widths_beyond_the_large_workload():
    """d = 8192, r = 1024, h = 2048: contractions twice as long and outputs twice as wide as the large workload's, on a
    batch small enough for the oracle (300 tokens, 4 experts)."""
    w = wl.Workload("wide", dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=211, T=300, d=8192, r=1024, h=2048, E=4, k=2)
    inp = conditioned(w)
    margin.enforce_margin(w, inp, 1e-3)
    compare_full(w, inp, run_full(w, inp))


@pytest.mark.parametrize("case", [
    # one expert takes a slot of nearly every token
    dict(shape=dict(T=6000, d=256, r=256, h=512, E=16, k=2), bias="one_hot"),
    # graded popularity: expert loads from thousands of rows down to none
    dict(shape=dict(T=6000, d=256, r=256, h=256, E=24, k=3), bias="graded"),
    # balanced, many row tiles per expert
    dict(shape=dict(T=20000, d=256, r=256, h=256, E=24, k=2), bias=None),
])
@pytest.mark.parametrize("flags", [0, wl.FLAG_DYNAMIC_WGRAD])
def test_bf16_skewed_routing(case, flags):
    """Expert-load skew (dropless routing keeps every slot, so one expert may hold most rows and others none):
    results must match the oracle as for balanced routing, also when accumulating into existing gradients; with
    the statically scheduled weight-gradient kernel (the default at these sizes) and the dynamically scheduled one
    that cuts long experts into parts."""
    import torch

    w = wl.Workload("skew", dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=311, **case["shape"])
    inp = conditioned(w)
    if case["bias"] == "one_hot":
        b = np.zeros(w.E, dtype=np.float32)
        b[3] = 8.0
        inp["b_gate"] = b
    elif case["bias"] == "graded":
        inp["b_gate"] = (2.5 * np.linspace(1.0, -1.0, w.E) ** 3).astype(np.float32)
    margin.enforce_margin(w, inp, 1e-3)
    got = run_full(w, inp, flags)
    compare_full(w, inp, got)
    if case["bias"] == "one_hot":
        assert got["routing"]["counts"][3].item() >= 0.9 * w.T
        dev = to_device(w, inp)
        layer = make_layer(w, flags)
        layer.forward(dev["x"], dev, training=True)
        G1 = empty_grads(w, "cuda", fill=0.5)
        layer.backward(dev["x"], dev["dy"], dev, G1, accumulate=True)
        torch.cuda.synchronize()
        for key in ("dw1", "dw2"):
            ref = got[key] + 0.5
            assert np.max(np.abs(to_numpy(G1[key]) - ref)) <= 2.0 ** -7 * np.max(np.abs(ref)), key
        layer.close()


@pytest.mark.parametrize("case", [
    dict(dtype=wl.DTYPE_F32, act=wl.ACT_GELU_ERF, T=77, d=36, h=20, E=5, k=2),
    dict(dtype=wl.DTYPE_F32, act=wl.ACT_RELU, T=300, d=64, h=8, E=7, k=3),
    dict(dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, T=1000, d=256, h=64, E=16, k=4),     # narrow experts: one-CTA kernels
    dict(dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, T=2048, d=1024, h=256, E=8, k=2),    # CTA pairs, staged stores
    dict(dtype=wl.DTYPE_BF16, act=wl.ACT_RELU, T=130, d=320, h=128, E=40, k=2),
])
def test_projection_free_layer_of_eq3(case):
    """BIGMAC_FLAG_CDAC: y = sum_i p_i(x) E_i(x) with d -> h -> d experts, dispatched at width d, forward and
    backward, against the oracle (which evaluates it as Eq. 2 with identity projections)."""
    case = dict(case)
    d = case.pop("d")
    w = wl.Workload("cdac", d=d, r=d, seed=577, cdac=True, **case)
    inp = conditioned(w)
    assert inp["w_down"] is None and inp["w_up"] is None
    compare_full(w, inp, run_full(w, inp))


def test_small_cdac_twin_full_config():
    """The parameter-parity twin of configs[1] (d=1024, E=32, k=4, experts 1024 -> 64 -> 1024) at T=2048."""
    w = wl.WORKLOADS["small"].cdac_twin().with_tokens(2048)
    assert (w.r, w.h, w.cdac) == (1024, 64, True)
    inp = conditioned(w)
    compare_full(w, inp, run_full(w, inp))


@pytest.mark.parametrize("shape", [
    dict(T=1, d=64, r=256, h=256, E=8, k=3),        # one token: most experts empty (their gradients are zero-filled)
    dict(T=333, d=128, r=320, h=256, E=5, k=5),     # ragged widths (320 = 256 + 64), k = E
    dict(T=4096, d=256, r=256, h=1024, E=4, k=1),   # few experts, thousands of rows each: every expert in parts
])
def test_bf16_dynamic_weight_gradient_kernel(shape):
    w = wl.Workload("dyn", dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=733, **shape)
    inp = conditioned(w)
    compare_full(w, inp, run_full(w, inp, wl.FLAG_DYNAMIC_WGRAD))


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


@pytest.mark.parametrize("T", [1, 3, 8, 16])
@pytest.mark.parametrize("shape", [
    dict(d=2048, r=256, h=1024, E=64, k=8),        # the decode configuration
    dict(d=192, r=64, h=320, E=5, k=5),            # k = E, ragged widths
    dict(d=64, r=128, h=64, E=40, k=1),
])
def test_small_batch_inference_forward(T, shape):
    """Inference forward at a handful of tokens (one fused kernel): y and the routing tables against the oracle."""
    import torch

    w = wl.Workload("decode", T=T, dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=300 + T, **shape)
    inp = conditioned(w)
    inp["b_gate"] = (np.linspace(-0.2, 0.2, w.E)).astype(np.float32)
    margin.enforce_margin(w, inp, 1e-3)
    dev = to_device(w, inp)
    layer = make_layer(w)
    y, R = layer.forward(dev["x"], dev, training=False, want_routing=True)
    y2 = layer.forward(dev["x"], dev, training=False)            # no tables requested: same kernel, same result
    torch.cuda.synchronize()
    assert layer.status() == 0
    rt = oracle.route(inp, w.k)
    check_routing(R, rt)
    ref = oracle.forward_tokens(inp, rt, w.act)["y"]
    assert_within(w, float_errors(w, {"y": to_numpy(y)}, {"y": ref}))
    assert torch.equal(y, y2)
    layer.close()


@pytest.mark.parametrize("T", [17, 64, 200, 512, 1024])
@pytest.mark.parametrize("shape", [
    dict(d=2048, r=256, h=1024, E=64, k=8),        # the decode configuration
    dict(d=512, r=128, h=256, E=12, k=3),          # four hidden chunks, two per CTA of a pair
])
def test_inference_forward_of_a_few_hundred_tokens(T, shape):
    """Inference forward above the one-kernel limit at decode-like sizes: the descend + logits contraction runs in
    parts (fp32 partial results, added by a small kernel) and the experts run on CTA pairs that share a tile's hidden
    chunks.  y and the routing tables against the oracle; two calls agree bit for bit."""
    import torch

    w = wl.Workload("decode", T=T, dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=700 + T, **shape)
    inp = conditioned(w)
    inp["b_gate"] = (np.linspace(-0.2, 0.2, w.E)).astype(np.float32)
    margin.enforce_margin(w, inp, 1e-3)
    dev = to_device(w, inp)
    layer = make_layer(w)
    y, R = layer.forward(dev["x"], dev, training=False, want_routing=True)
    y2 = layer.forward(dev["x"], dev, training=False)
    torch.cuda.synchronize()
    assert layer.status() == 0
    rt = oracle.route(inp, w.k)
    check_routing(R, rt)
    ref = oracle.forward_tokens(inp, rt, w.act)["y"]
    assert_within(w, float_errors(w, {"y": to_numpy(y)}, {"y": ref}))
    assert torch.equal(y, y2)
    layer.close()


@pytest.mark.parametrize("case", [
    dict(T=300, d=128, r=64, h=192, E=5, k=2, act=wl.ACT_GELU_ERF),      # narrowest width, three hidden chunks, ragged segments
    dict(T=1000, d=256, r=192, h=320, E=16, k=4, act=wl.ACT_RELU),       # widths that are odd multiples of 64
    dict(T=2048, d=512, r=256, h=1024, E=8, k=2, act=wl.ACT_GELU_ERF),   # the widest case: all of shared memory, 384 TMEM columns
    dict(T=700, d=128, r=128, h=64, E=40, k=1, act=wl.ACT_GELU_TANH),    # one hidden chunk per tile, empty experts
])
def test_inference_forward_with_the_experts_in_one_kernel(case):
    """Inference forward above the small-batch limit with r <= 256: expert GEMM1, sigma and GEMM2 run as one kernel
    whose hidden activations stay on the SM.  y against the oracle, and against the training forward of the same
    layer (which stores the activations in HBM)."""
    import torch

    case = dict(case)
    act = case.pop("act")
    w = wl.Workload("mlp", dtype=wl.DTYPE_BF16, act=act, seed=911, **case)
    inp = conditioned(w)
    dev = to_device(w, inp)
    layer = make_layer(w)
    y, R = layer.forward(dev["x"], dev, training=False, want_routing=True)
    y_train = layer.forward(dev["x"], dev, training=True).clone()
    torch.cuda.synchronize()
    assert layer.status() == 0
    rt = oracle.route(inp, w.k)
    check_routing(R, rt)
    ref = oracle.forward_tokens(inp, rt, w.act)["y"]
    assert_within(w, float_errors(w, {"y": to_numpy(y)}, {"y": ref}))
    # same roundings (bf16 activations, fp32 accumulation), different accumulation grouping only
    assert oracle.max_rel_err(to_numpy(y), to_numpy(y_train)) <= 2.0 ** -7
    layer.close()


@pytest.mark.parametrize("T,E,k", [(1, 1, 1), (31, 7, 1), (128, 256, 8), (1024, 5, 1), (205, 64, 5), (256, 256, 8),
                                   (2048, 3, 1), (257, 16, 8), (683, 40, 3), (300, 300, 7),
                                   (150000, 64, 8), (70000, 1024, 4)])
@pytest.mark.parametrize("f", [0.0, 0.7])
def test_routing_tables_around_the_single_block_limit(T, E, k, f):
    """Up to 2048 slots and 256 experts the tables come from one single-block kernel (one or two chunks of 1024
    slots), beyond from the three-pass sort: both sides of both limits, with and without a capacity limit; and two
    batches well beyond the large workload's (1.2 million slots; 1024 experts), every table bit for bit."""
    import torch

    w = wl.Workload("tb", T=T, d=32, r=8, h=8, E=E, k=k, dtype=wl.DTYPE_F32, act=wl.ACT_RELU, seed=157)
    inp = conditioned(w)
    inp["b_gate"] = (2.0 * np.linspace(1.0, -1.0, E) ** 3).astype(np.float32)
    margin.enforce_margin(w, inp, 1e-3)
    dev = to_device(w, inp)
    layer = make_layer(w, capacity_factor=f)
    R = layer.route(dev["x"], dev)
    torch.cuda.synchronize()
    assert layer.status() == 0
    check_routing(R, oracle.route(inp, w.k, capacity_factor=f))
    layer.close()


@pytest.mark.parametrize("case", [
    dict(T=300, d=128, r=64, h=192, E=5, k=2, act=wl.ACT_GELU_ERF),       # one k slice per tile, ragged segments, narrow outputs
    dict(T=1000, d=256, r=320, h=1024, E=16, k=4, act=wl.ACT_RELU),       # five k slices: more than the gather's lag, staged stores
    dict(T=5000, d=512, r=512, h=2048, E=8, k=2, act=wl.ACT_GELU_ERF),    # the large workload's widths, many row tiles per SM
    dict(T=700, d=128, r=128, h=64, E=40, k=1, act=wl.ACT_GELU_TANH),     # empty experts, 128-wide tiles
    dict(T=2, d=64, r=64, h=256, E=8, k=3, act=wl.ACT_GELU_ERF),          # nearly all padding rows
])
def test_inference_forward_with_the_dispatch_fused_into_expert_gemm1(case):
    """Inference forward with the two expert GEMMs as separate launches: expert GEMM1 gathers the rows of x' itself
    (no grouped copy is written).  y against the oracle, and bit for bit against the same forward with the standalone
    dispatch kernel in front (same operands, same arithmetic order)."""
    import torch
    from paper_2502_16927_b200 import binding

    case = dict(case)
    act = case.pop("act")
    w = wl.Workload("fd", dtype=wl.DTYPE_BF16, act=act, seed=977, **case)
    inp = conditioned(w)
    dev = to_device(w, inp)
    binding.bigmac_debug_set("fused_mlp", 0)
    binding.bigmac_debug_set("fuse_dispatch", 1)
    try:
        layer = make_layer(w)
        y, R = layer.forward(dev["x"], dev, training=False, want_routing=True)
        y = y.clone()
        binding.bigmac_debug_set("fuse_dispatch", 0)
        y_plain = layer.forward(dev["x"], dev, training=False).clone()
        torch.cuda.synchronize()
        assert layer.status() == 0
        layer.close()
    finally:
        binding.bigmac_debug_set("defaults")
    rt = oracle.route(inp, w.k)
    check_routing(R, rt)
    assert_within(w, float_errors(w, {"y": to_numpy(y)}, {"y": oracle.forward_tokens(inp, rt, w.act)["y"]}))
    assert torch.equal(y.view(torch.int16), y_plain.view(torch.int16))


@pytest.mark.parametrize("case", [
    dict(shape=dict(T=6000, d=256, r=256, h=512, E=16, k=2), bias="graded", flags=wl.FLAG_DYNAMIC_WGRAD),   # long and empty experts, parts
    dict(shape=dict(T=333, d=128, r=384, h=256, E=5, k=5), bias=None, flags=wl.FLAG_DYNAMIC_WGRAD),         # ragged widths (384 = 256 + 128), k = E
    dict(shape=dict(T=20000, d=256, r=256, h=256, E=24, k=2), bias=None, flags=wl.FLAG_DYNAMIC_WGRAD),      # balanced, many row tiles per expert
    dict(shape=dict(T=9000, d=512, r=512, h=1024, E=8, k=4), bias=None, flags=0),                           # enough work for the balanced kernel by size
])
def test_training_step_with_the_dispatch_fused_into_its_consumers(case):
    """Training forward + backward without a grouped copy of x': expert GEMM1 and the weight gradient dW1 gather the
    rows of x' themselves.  Every output against the oracle, and bit for bit against the same step with the standalone
    dispatch kernel (same operands, same arithmetic order)."""
    import torch
    from paper_2502_16927_b200 import binding

    w = wl.Workload("fdt", dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=983, **case["shape"])
    inp = conditioned(w)
    if case["bias"] == "graded":
        inp["b_gate"] = (2.5 * np.linspace(1.0, -1.0, w.E) ** 3).astype(np.float32)
        margin.enforce_margin(w, inp, 1e-3)
    binding.bigmac_debug_set("fuse_dispatch", 1)
    try:
        got = run_full(w, inp, case["flags"])
        compare_full(w, inp, got)
        prof_layer = make_layer(w, case["flags"])
        dev = to_device(w, inp)
        binding.bigmac_profile_enable(prof_layer.handle, True)
        prof_layer.forward(dev["x"], dev, training=True)
        stages = binding.bigmac_profile_read(prof_layer.handle)["stages"]
        binding.bigmac_profile_enable(prof_layer.handle, False)
        prof_layer.close()
        assert "dispatch" not in stages, stages            # the fused path ran: no dispatch launch in the forward
    finally:
        binding.bigmac_debug_set("defaults")
    plain = run_full(w, inp, case["flags"])
    for key in ("y", "dx", "dw1", "dw2", "dw_up", "dw_down", "dw_gate", "db_gate"):
        np.testing.assert_array_equal(got[key], plain[key], err_msg=key)
