"""GPU parity of the expert-bias variant (BIGMAC_FLAG_EXPERT_BIAS: z = x' W1^T + b1, u = sigma(z) W2^T + b2, fp32
biases and bias gradients) against the CPU oracle."""
import numpy as np
import pytest

import oracle
from oracle import margin
from paper_2502_16927_b200 import binding, workloads as wl

from helpers import make_layer, oracle_inputs, to_device, to_numpy
from test_gpu_parity import BF16_FRO, TOL, compare_full, conditioned, run_full

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape", [
    dict(T=500, d=64, r=24, h=40, E=10, k=3),
    dict(T=129, d=32, r=8, h=20, E=7, k=7),
    dict(T=1, d=16, r=8, h=8, E=4, k=1),
])
@pytest.mark.parametrize("act", [wl.ACT_GELU_ERF, wl.ACT_RELU, wl.ACT_GELU_TANH])
def test_fp32_expert_biases(shape, act):
    w = wl.Workload("eb", dtype=wl.DTYPE_F32, act=act, seed=101, expert_bias=True, **shape)
    inp = conditioned(w)
    compare_full(w, inp, run_full(w, inp))


@pytest.mark.parametrize("shape", [
    dict(T=3000, d=256, r=128, h=256, E=16, k=4),
    dict(T=2000, d=256, r=256, h=1024, E=8, k=2),     # staged stores in both expert GEMMs
    dict(T=1500, d=128, r=64, h=128, E=24, k=3),      # experts without rows, narrow outputs
])
@pytest.mark.parametrize("flags", [0, wl.FLAG_SIMT_GEMM])
def test_bf16_expert_biases(shape, flags):
    w = wl.Workload("eb", dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=103, expert_bias=True, **shape)
    inp = conditioned(w)
    inp["b_gate"] = (2.0 * np.linspace(1.0, -1.0, w.E) ** 3).astype(np.float32)
    margin.enforce_margin(w, inp, 1e-3)
    compare_full(w, inp, run_full(w, inp, flags))


def test_small_config_with_expert_biases():
    w = wl.Workload(**{**wl.WORKLOADS["small"].__dict__, "expert_bias": True})
    inp = conditioned(w)
    compare_full(w, inp, run_full(w, inp))


def test_eq3_layer_and_capacity_limit_with_expert_biases():
    w = wl.Workload("eb", T=2000, d=128, r=128, h=64, E=8, k=2, dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=107, cdac=True,
                    expert_bias=True)
    inp = conditioned(w)
    compare_full(w, inp, run_full(w, inp))
    w2 = wl.Workload("eb", T=700, d=64, r=24, h=40, E=10, k=3, dtype=wl.DTYPE_F32, act=wl.ACT_GELU_ERF, seed=109, expert_bias=True)
    inp2 = conditioned(w2)
    inp2["b_gate"] = (1.5 * np.linspace(1.0, -1.0, w2.E) ** 3).astype(np.float32)
    margin.enforce_margin(w2, inp2, 1e-3)
    compare_full(w2, inp2, run_full(w2, inp2, capacity_factor=0.6), capacity_factor=0.6)


@pytest.mark.parametrize("T", [4, 300])
def test_inference_forward_with_expert_biases(T):
    """Few tokens and short tile lists: the one-kernel decode forward and the fused expert kernel are bypassed."""
    import torch

    w = wl.Workload("eb", T=T, d=256, r=128, h=256, E=16, k=4, dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=113, expert_bias=True)
    inp = conditioned(w)
    rt = oracle.route(inp, w.k)
    ref = oracle.forward_tokens(inp, rt, w.act)["y"]
    dev = to_device(w, inp)
    layer = make_layer(w)
    y = layer.forward(dev["x"], dev, training=False)
    torch.cuda.synchronize()
    assert layer.status() == 0
    assert oracle.max_rel_err(to_numpy(y), ref) <= TOL[w.dtype] and oracle.fro_rel_err(to_numpy(y), ref) <= (BF16_FRO if w.dtype == wl.DTYPE_BF16 else TOL[w.dtype])
    layer.close()


def test_biases_are_required_with_the_flag_and_rejected_for_expert_parallel_handles():
    import torch

    w = wl.Workload("eb", T=64, d=64, r=24, h=40, E=10, k=3, dtype=wl.DTYPE_F32, act=wl.ACT_GELU_ERF, seed=127, expert_bias=True)
    inp = conditioned(w)
    dev = to_device(w, inp)
    layer = make_layer(w)
    missing = {key: val for key, val in dev.items() if key != "b2"}
    with pytest.raises(binding.BigmacError) as err:
        layer.forward(dev["x"], missing)
    assert err.value.status == -1
    with pytest.raises(binding.BigmacError) as err:
        binding.bigmac_ep_buffer_bytes(layer.handle, 2)
    assert err.value.status == -2
    layer.close()
