"""Seeded random configurations of the layer and its variants (dtype, shapes that are not multiples of any tile size,
expert counts, k, activation, gate skew; the Eq. 3 layer, the gate on x', expert biases, a capacity limit, the
load-balancing loss; tensor-core and FMA contractions, both weight-gradient kernels) against the CPU oracle, with the
comparison rules of test_gpu_parity.py.  The same generator ran several hundred further configurations while the
kernels were written; these forty are the regression sample."""
import numpy as np
import pytest

from oracle import margin
from paper_2502_16927_b200 import workloads as wl

import test_gpu_gate_low as gate_low_cases
import test_gpu_parity as parity

pytestmark = pytest.mark.gpu

VARIANTS = ("plain", "cdac", "gate_low", "bias", "cap", "aux", "cap_aux", "bias_cap")


def draw(seed):
    rng = np.random.default_rng(seed)
    bf16 = rng.random() < 0.6
    if bf16:
        d, r, h = (int(rng.choice(c)) for c in ([64, 128, 192, 256, 320], [64, 128, 192, 256], [64, 128, 192, 256, 512, 1024]))
        T = int(rng.integers(1, 4000))
    else:
        d, r, h = 4 * int(rng.integers(2, 24)), 4 * int(rng.integers(1, 12)), 4 * int(rng.integers(1, 16))
        T = int(rng.integers(1, 700))
    variant = VARIANTS[seed % len(VARIANTS)]
    E = int(rng.integers(1, 40 if variant == "gate_low" else 130))
    k = int(rng.integers(1, min(E, 8 if variant == "gate_low" else 14) + 1))
    act = int(rng.choice([wl.ACT_RELU, wl.ACT_GELU_ERF] if bf16 else [wl.ACT_RELU, wl.ACT_GELU_ERF, wl.ACT_GELU_TANH]))
    kw, run_kw = dict(cdac=False, gate_low=False, expert_bias=False), {}
    if variant == "cdac":
        kw["cdac"], r = True, d
    kw["gate_low"] = variant == "gate_low"
    kw["expert_bias"] = variant in ("bias", "bias_cap")
    if variant in ("cap", "cap_aux", "bias_cap"):
        run_kw["capacity_factor"] = float(rng.choice([0.3, 0.8, 1.0, 1.2, 2.0]))
    if variant in ("aux", "cap_aux"):
        run_kw["aux"] = float(rng.choice([0.001, 1.0, 30.0]))
    flags = int(rng.choice([0, 0, wl.FLAG_DYNAMIC_WGRAD, wl.FLAG_SIMT_GEMM])) if bf16 else 0
    skew = float(rng.choice([0.0, 1.0, 3.0]))
    w = wl.Workload("rnd", T=T, d=d, r=r, h=h, E=E, k=k, dtype=wl.DTYPE_BF16 if bf16 else wl.DTYPE_F32, act=act,
                    seed=9000 + seed, **kw)
    return w, run_kw, flags, skew


@pytest.mark.parametrize("seed", range(40))
def test_random_configuration(seed):
    w, run_kw, flags, skew = draw(seed)
    inp = wl.make_inputs(w)
    if skew:
        inp["b_gate"] = (skew * np.linspace(1.0, -1.0, w.E) ** 3).astype(np.float32)
    if w.gate_low:
        bf16 = w.dtype == wl.DTYPE_BF16
        margin.enforce_margin(w, inp, 2e-2 if bf16 else 1e-3, gate_low=True, round_x_lo_bf16=bf16)
        gate_low_cases.compare(w, inp, parity.run_full(w, inp, flags))
        return
    margin.enforce_margin(w, inp, 1e-3)
    cf, aux = run_kw.get("capacity_factor", 0.0), run_kw.get("aux", 0.0)
    parity.compare_full(w, inp, parity.run_full(w, inp, flags, capacity_factor=cf, aux=aux), capacity_factor=cf, aux=aux)
