"""Shared test helpers (CPU side): small grid-valued workloads for the oracle's pins."""
from __future__ import annotations

import numpy as np

from paper_2502_16927_b200 import workloads as wl


def small_workload(T=24, d=16, r=8, h=12, E=4, k=2, act=wl.ACT_GELU_ERF, seed=7, bias=False, grid=2.0 ** -10):
    """A tiny fp32 workload whose values lie on a coarse binary grid (so that +-delta perturbations
    used by finite differences stay exactly representable in float32)."""
    w = wl.Workload("t", T=T, d=d, r=r, h=h, E=E, k=k, dtype=wl.DTYPE_F32, act=act, seed=seed)
    inp = wl.make_inputs(w)
    for key, val in inp.items():
        if val is not None:
            inp[key] = (np.round(val / grid) * grid).astype(np.float32)
    if bias:
        g = np.random.default_rng(seed)
        inp["b_gate"] = (np.round(g.standard_normal(E) * 0.5 / grid) * grid).astype(np.float32)
    return w, inp


def regrid(w, inp, grid=2.0 ** -10):
    inp["x"] = (np.round(inp["x"] / grid) * grid).astype(np.float32)
