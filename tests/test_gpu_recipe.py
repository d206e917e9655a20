"""GPU parity of the training-recipe variants (Table 5: capacity factor, load-balancing loss): the CUDA layer,
through the C ABI, against the CPU oracle on the same seeded inputs.  Tables bit for bit (dropped slots are -1 on
both sides), floats within the tolerances of test_gpu_parity.py.  The loss coefficient is taken far above the
paper's 0.001 in most cases so that its gradient is as large as the layer's own and an error in it cannot hide."""
import numpy as np
import pytest

import oracle
from oracle import margin
from paper_2502_16927_b200 import binding, workloads as wl

from helpers import empty_grads, make_layer, to_device, to_numpy
from test_gpu_parity import BF16_FRO, TOL, check_routing, compare_full, conditioned, run_full

pytestmark = pytest.mark.gpu


def skewed(w, strength=1.5):
    inp = conditioned(w)
    inp["b_gate"] = (strength * np.linspace(1.0, -1.0, w.E) ** 3).astype(np.float32)
    margin.enforce_margin(w, inp, 1e-3)
    return inp


@pytest.mark.parametrize("f", [1.0, 0.5, 0.05, 1000.0])
@pytest.mark.parametrize("act", [wl.ACT_RELU, wl.ACT_GELU_ERF])
def test_fp32_capacity_factor(f, act):
    w = wl.Workload("cap", T=700, d=64, r=24, h=40, E=10, k=3, dtype=wl.DTYPE_F32, act=act, seed=41)
    inp = skewed(w)
    got = run_full(w, inp, capacity_factor=f)
    compare_full(w, inp, got, capacity_factor=f)
    ros = to_numpy(got["routing"]["row_of_slot"])
    if f < 1000.0:
        assert (ros < 0).any() and (ros >= 0).any()
    else:
        assert (ros >= 0).all()


@pytest.mark.parametrize("case", [
    dict(shape=dict(T=6000, d=256, r=256, h=512, E=16, k=2), strength=3.0, f=1.2),
    dict(shape=dict(T=6000, d=256, r=128, h=256, E=24, k=3), strength=2.0, f=1.0),
    dict(shape=dict(T=3000, d=128, r=64, h=128, E=8, k=2), strength=0.0, f=1.2),      # balanced: few drops
])
@pytest.mark.parametrize("flags", [0, wl.FLAG_DYNAMIC_WGRAD])
def test_bf16_capacity_factor(case, flags):
    w = wl.Workload("cap", dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=43, **case["shape"])
    inp = skewed(w, case["strength"])
    got = run_full(w, inp, flags, capacity_factor=case["f"])
    compare_full(w, inp, got, capacity_factor=case["f"])
    cap = oracle.capacity_rows(w.T, w.k, w.E, case["f"])
    assert to_numpy(got["routing"]["counts"]).max() <= cap


@pytest.mark.parametrize("alpha", [0.001, 40.0])
@pytest.mark.parametrize("bias", [False, True])
def test_fp32_aux_loss_value_and_its_gradient_alone(alpha, bias):
    """dy = 0: what the backward returns is the gradient of the load-balancing loss alone."""
    w = wl.Workload("aux", T=900, d=48, r=16, h=24, E=12, k=2, dtype=wl.DTYPE_F32, act=wl.ACT_GELU_ERF, seed=47)
    inp = skewed(w) if bias else conditioned(w)
    inp["dy"] = np.zeros_like(inp["dy"])
    got = run_full(w, inp, aux=alpha)
    compare_full(w, inp, got, aux=alpha)
    assert np.abs(got["dx"]).max() > 0 and np.abs(got["db_gate"]).max() > 0


@pytest.mark.parametrize("shape", [
    dict(T=900, d=48, r=16, h=24, E=12, k=2),
    dict(T=333, d=32, r=8, h=16, E=70, k=5),        # E not a multiple of 32, more than two experts per lane
    dict(T=50, d=32, r=8, h=16, E=3, k=3),          # fewer tokens than warps in the loss kernels
])
def test_fp32_aux_loss_with_the_layer_gradient(shape):
    w = wl.Workload("aux", dtype=wl.DTYPE_F32, act=wl.ACT_GELU_TANH, seed=53, **shape)
    inp = skewed(w)
    got = run_full(w, inp, aux=25.0)
    compare_full(w, inp, got, aux=25.0)


@pytest.mark.parametrize("flags", [0, wl.FLAG_SIMT_GEMM])
def test_small_bf16_with_the_pre_training_recipe(flags):
    """The small configuration with Table 5's settings (capacity factor 1.2, loss coefficient 0.001) and, so that the
    loss gradient is visible in BF16, with a coefficient of 2000."""
    w = wl.WORKLOADS["small"]
    inp = skewed(w, 1.0)
    for alpha in (0.001, 2000.0):
        got = run_full(w, inp, flags, capacity_factor=1.2, aux=alpha)
        compare_full(w, inp, got, capacity_factor=1.2, aux=alpha)


def test_cdac_layer_with_capacity_and_aux_loss():
    w = wl.Workload("cap", T=2000, d=128, r=128, h=64, E=8, k=2, dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=59, cdac=True)
    inp = skewed(w, 2.0)
    got = run_full(w, inp, capacity_factor=1.0, aux=500.0)
    compare_full(w, inp, got, capacity_factor=1.0, aux=500.0)


@pytest.mark.parametrize("T", [8, 300, 5000])
def test_inference_forward_and_route_under_a_capacity_limit(T):
    """The inference forward (few tokens: the general path instead of the one-kernel decode forward; short tile
    lists: the experts in one kernel) and the routing-only entry points drop the same slots."""
    import torch

    w = wl.Workload("cap", T=T, d=256, r=128, h=256, E=16, k=4, dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=61)
    inp = skewed(w, 2.0)
    f, alpha = 0.75, 3.0
    rt = oracle.route(inp, w.k, capacity_factor=f)
    ref = oracle.forward_tokens(inp, rt, w.act)["y"]
    loss = oracle.aux_loss(rt.logits, rt.topk_idx, alpha, want_grad=False)[0]
    dev = to_device(w, inp)
    layer = make_layer(w, capacity_factor=f, aux_loss_coef=alpha)
    y, R = layer.forward(dev["x"], dev, training=False, want_routing=True)
    R2 = layer.route(dev["x"], dev)
    R3 = layer.empty_routing(T)
    binding.bigmac_route_static(layer.handle, dev["x"], T, dev, R3)
    torch.cuda.synchronize()
    assert layer.status() == 0
    for tables in (R, R2, R3):
        check_routing(tables, rt)
        assert abs(tables["aux_loss"].item() - loss) <= 1e-5 * loss
    assert oracle.max_rel_err(to_numpy(y), ref) <= TOL[w.dtype]
    assert oracle.fro_rel_err(to_numpy(y), ref) <= (BF16_FRO if w.dtype == wl.DTYPE_BF16 else TOL[w.dtype])
    layer.close()


def test_accumulate_with_capacity_and_aux_loss_adds_to_existing_gradients():
    import torch

    w = wl.Workload("cap", T=700, d=64, r=24, h=40, E=10, k=3, dtype=wl.DTYPE_F32, act=wl.ACT_GELU_ERF, seed=67)
    inp = skewed(w)
    base = run_full(w, inp, capacity_factor=0.5, aux=10.0)
    dev = to_device(w, inp)
    layer = make_layer(w, capacity_factor=0.5, aux_loss_coef=10.0)
    layer.forward(dev["x"], dev, training=True)
    G = empty_grads(w, "cuda", fill=0.25)
    layer.backward(dev["x"], dev["dy"], dev, G, accumulate=True)
    torch.cuda.synchronize()
    for key, val in G.items():
        ref = base[key] + 0.25
        assert np.max(np.abs(to_numpy(val) - ref)) <= 1e-5 * np.max(np.abs(ref)), key
    layer.close()


def test_recipe_settings_are_validated():
    w = wl.WORKLOADS["tiny"]
    for kw in (dict(capacity_factor=-1.0), dict(aux_loss_coef=-0.5), dict(capacity_factor=float("nan")),
               dict(aux_loss_coef=float("inf"))):
        with pytest.raises(binding.BigmacError) as err:
            make_layer(w, **kw)
        assert err.value.status == -1
