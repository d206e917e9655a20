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


# ---------------------------------------------------------------------------------------------
# GPU side: move a generated workload to the device and run it through the C ABI binding.
# ---------------------------------------------------------------------------------------------

def to_device(w, inp, device="cuda"):
    """numpy float32 arrays (dtype-representable values) -> torch tensors of the workload dtype."""
    import torch

    out = {}
    for key, val in inp.items():
        if val is None:
            continue
        if key in ("b_gate", "b1", "b2") or w.dtype == wl.DTYPE_F32:
            out[key] = torch.from_numpy(np.ascontiguousarray(val, dtype=np.float32)).to(device)
        else:
            bits = torch.from_numpy(wl.to_bf16_bits(val).view(np.int16)).to(device)
            out[key] = bits.view(torch.bfloat16)
    return out


def to_numpy(t):
    """torch tensor (fp32 / bf16 / int32) -> numpy float64 or int32."""
    import torch

    if t.dtype in (torch.int32, torch.int64):
        return t.cpu().numpy()
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def make_layer(w, flags=0, max_tokens=None, capacity_factor=0.0, aux_loss_coef=0.0):
    from paper_2502_16927_b200 import binding

    if w.cdac:
        flags |= wl.FLAG_CDAC
    if w.gate_low:
        flags |= wl.FLAG_GATE_LOW
    if w.expert_bias:
        flags |= wl.FLAG_EXPERT_BIAS
    return binding.Layer(w.d, w.r, w.h, w.E, w.k, max_tokens or max(w.T, 1), w.dtype, w.act, flags,
                         capacity_factor=capacity_factor, aux_loss_coef=aux_loss_coef)


def oracle_inputs(w, inp):
    """What the oracle is given for this workload.  The projection-free layer (Eq. 3) is Eq. 2 with identity
    projections, which is how the oracle evaluates it."""
    if not w.cdac:
        return inp
    out = dict(inp)
    out["w_down"] = np.eye(w.d, dtype=np.float32)
    out["w_up"] = np.eye(w.d, dtype=np.float32)
    return out


def empty_grads(w, dev, fill=None):
    import torch

    dt = torch.float32 if w.dtype == wl.DTYPE_F32 else torch.bfloat16
    shapes = {"dw_gate": (w.E, w.r if w.gate_low else w.d), "dw_down": (w.r, w.d), "dw1": (w.E, w.h, w.r), "dw2": (w.E, w.r, w.h),
              "dw_up": (w.d, w.r)}
    if w.cdac:
        del shapes["dw_down"], shapes["dw_up"]
    G = {}
    for key, shp in shapes.items():
        G[key] = torch.empty(shp, dtype=dt, device="cuda") if fill is None else torch.full(shp, fill, dtype=dt, device="cuda")
    f32 = {"db_gate": (w.E,)}
    if w.expert_bias:
        f32.update(db1=(w.E, w.h), db2=(w.E, w.r))
    for key, shp in f32.items():
        G[key] = (torch.empty(shp, dtype=torch.float32, device="cuda") if fill is None
                  else torch.full(shp, fill, dtype=torch.float32, device="cuda"))
    return G
