"""GPU parity of the gate-on-x' variant (BIGMAC_FLAG_GATE_LOW: logits from the low-width token, w_gate [E,r]) against
the CPU oracle.  In BF16 the kernels read x' as stored (bf16), so the oracle rounds x' to bf16 before the gate too:
the top-k decision is taken on the same numbers on both sides."""
import numpy as np
import pytest

import oracle
from oracle import margin
from paper_2502_16927_b200 import binding, workloads as wl

from helpers import make_layer, to_device, to_numpy
from test_gpu_parity import RELU_DECISION_KEYS, RELU_OUTLIER, TOL, assert_within, check_routing, float_errors, outlier_fraction, run_full

pytestmark = pytest.mark.gpu


def conditioned(w, strength=0.0):
    inp = wl.make_inputs(w)
    if strength:
        inp["b_gate"] = (strength * np.linspace(1.0, -1.0, w.E) ** 3).astype(np.float32)
    margin.enforce_margin(w, inp, 1e-3 if w.dtype == wl.DTYPE_F32 else 2e-2, gate_low=True,
                          round_x_lo_bf16=w.dtype == wl.DTYPE_BF16)
    return inp


# Gate values in BF16: the kernels round the fp32-accumulated x' to bf16, the oracle the exact x'; an element that sits
# next to a rounding boundary lands on the other neighbour (2^-8 relative), which moves a logit by up to about
# 2^-8 |x'_c W_g[e,c]| ~ 4e-4 and a gate value by a quarter of that per such element.  The integer tables are still
# compared bit for bit (the inputs are conditioned to a top-k margin of 2e-2).
P_ATOL = {wl.DTYPE_F32: 2e-5, wl.DTYPE_BF16: 1e-3}


def compare(w, inp, got, capacity_factor=0.0):
    bf16 = w.dtype == wl.DTYPE_BF16
    rt = oracle.route(inp, w.k, capacity_factor=capacity_factor, gate_low=True, round_x_lo_bf16=bf16)
    check_routing(got["routing"], rt, P_ATOL[w.dtype])
    ref = oracle.backward_full(inp, rt, w.act, decide_bf16=bf16)
    ref["dw1"] = np.stack([ref["dw1"][e] for e in range(w.E)])
    ref["dw2"] = np.stack([ref["dw2"][e] for e in range(w.E)])
    keys = ("y", "dx", "dw_gate", "dw1", "dw2", "db_gate", "dw_up", "dw_down")
    assert got["dw_gate"].shape == (w.E, w.r)
    errs = float_errors(w, {key: got[key] for key in keys}, ref)
    if bf16 and w.act == wl.ACT_RELU:                  # isolated ReLU' decisions inside the accumulation noise (see test_gpu_parity)
        for key in RELU_DECISION_KEYS:
            if key in keys:
                assert outlier_fraction(got[key], ref[key], RELU_OUTLIER) <= 1e-3, key
                errs.pop(key)
                errs.pop(key + ":rms")
    assert_within(w, errs)


@pytest.mark.parametrize("shape", [
    dict(T=500, d=64, r=24, h=40, E=10, k=3),
    dict(T=129, d=32, r=8, h=16, E=70, k=5),
])
@pytest.mark.parametrize("act", [wl.ACT_GELU_ERF, wl.ACT_RELU])
def test_fp32_gate_on_the_low_width_token(shape, act):
    w = wl.Workload("gl", dtype=wl.DTYPE_F32, act=act, seed=83, gate_low=True, **shape)
    inp = conditioned(w, 1.0)
    compare(w, inp, run_full(w, inp))


@pytest.mark.parametrize("shape", [
    dict(T=3000, d=256, r=128, h=256, E=16, k=4),
    dict(T=2000, d=256, r=256, h=512, E=8, k=2),
    dict(T=1500, d=128, r=64, h=128, E=24, k=3),
])
@pytest.mark.parametrize("flags", [0, wl.FLAG_SIMT_GEMM])
@pytest.mark.parametrize("act", [wl.ACT_GELU_ERF, wl.ACT_RELU])
def test_bf16_gate_on_the_low_width_token(shape, flags, act):
    w = wl.Workload("gl", dtype=wl.DTYPE_BF16, act=act, seed=89, gate_low=True, **shape)
    inp = conditioned(w, 1.0)
    compare(w, inp, run_full(w, inp, flags))


def test_gate_on_the_low_width_token_with_a_capacity_limit_and_the_other_entry_points():
    import torch

    w = wl.Workload("gl", T=900, d=64, r=24, h=40, E=10, k=3, dtype=wl.DTYPE_F32, act=wl.ACT_GELU_ERF, seed=97, gate_low=True)
    inp = conditioned(w, 1.5)
    compare(w, inp, run_full(w, inp, capacity_factor=0.6), capacity_factor=0.6)
    rt = oracle.route(inp, w.k, gate_low=True)
    ref = oracle.forward_tokens(inp, rt, w.act)["y"]
    dev = to_device(w, inp)
    layer = make_layer(w)
    y, R = layer.forward(dev["x"], dev, training=False, want_routing=True)
    R2 = layer.route(dev["x"], dev)
    R3 = layer.empty_routing(w.T)
    binding.bigmac_route_static(layer.handle, dev["x"], w.T, dev, R3)
    torch.cuda.synchronize()
    assert layer.status() == 0
    for tables in (R, R2, R3):
        check_routing(tables, rt)
    assert_within(w, float_errors(w, {"y": to_numpy(y)}, {"y": ref}))
    layer.close()


def test_flag_combinations_are_validated():
    w = wl.WORKLOADS["tiny"]
    with pytest.raises(binding.BigmacError) as err:
        binding.Layer(w.d, w.d, w.h, w.E, w.k, 64, w.dtype, w.act, wl.FLAG_GATE_LOW | wl.FLAG_CDAC)
    assert err.value.status == -1
    with pytest.raises(binding.BigmacError) as err:
        binding.Layer(w.d, w.r, w.h, w.E, w.k, 64, w.dtype, w.act, wl.FLAG_GATE_LOW, aux_loss_coef=0.1)
    assert err.value.status == -2
