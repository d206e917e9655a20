"""Seeded synthetic inputs for the BigMac DCCA MoE layer.

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the layer's arithmetic: it only names the workload shapes and draws
random tensors.  Everything is generated with numpy's counter-based Philox
generator keyed by (seed, tensor tag, attempt), so any tensor can be drawn
independently of the others.

Shapes follow the GPT-3-style MoE workloads the paper measures (sequence
length 2048, hidden widths 1024 / 2048 / 4096, 64 experts with top-4 / top-8
routing, BF16); the data are synthetic stand-ins for its text corpora, because
the cost of the layer depends only on shapes and on the routing histogram.

Notation (paper's Table 2 in brackets): T tokens [b*s], d model width [h],
r low width in which tokens travel [r*h], h expert hidden width, E experts [e],
k experts per token [top_k].

All float tensors are returned as float32 arrays whose values are exactly
representable in the workload's dtype (bf16 values are a subset of fp32), so
both sides start from bit-identical numbers.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import os

import numpy as np

ACT_RELU, ACT_GELU_ERF, ACT_GELU_TANH, ACT_IDENTITY = 0, 1, 2, 3
DTYPE_F32, DTYPE_BF16 = 0, 1
FLAG_SIMT_GEMM, FLAG_CDAC, FLAG_DYNAMIC_WGRAD, FLAG_GATE_LOW, FLAG_EXPERT_BIAS = 1, 2, 4, 8, 16


@dataclass(frozen=True)
class Workload:
    name: str
    T: int
    d: int
    r: int
    h: int
    E: int
    k: int
    dtype: int
    act: int
    seed: int
    gate_bias: str = "none"   # "none" | "zipf"  (b_g[e] = ln q_e, q_e ~ (e+1)^-1.1)
    cdac: bool = False        # the conventional fine-grained layer (Eq. 3): r == d, no w_down / w_up
    gate_low: bool = False    # the gate reads x' (w_gate [E,r]) instead of x
    expert_bias: bool = False # experts have fp32 biases b1 [E,h], b2 [E,r] ~ N(0, 0.25)

    @property
    def N(self) -> int:
        return self.T * self.k

    def with_tokens(self, T: int, seed: Optional[int] = None) -> "Workload":
        return replace(self, T=T, seed=self.seed if seed is None else seed)

    def cdac_twin(self) -> "Workload":
        """The conventional fine-grained MoE layer with the same E, k, d and the same number of expert
        parameters: experts d -> m -> d with m = r h / d (the paper's parameter-parity rule), tokens
        dispatched at width d."""
        assert not self.cdac and (self.r * self.h) % self.d == 0
        return replace(self, name=self.name + "_cdac", r=self.d, h=self.r * self.h // self.d, cdac=True)


# The five configurations the layer is built and measured on.
WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", T=256, d=128, r=32, h=128, E=8, k=2,
                     dtype=DTYPE_F32, act=ACT_RELU, seed=1234),
    "small": Workload("small", T=4096, d=1024, r=128, h=512, E=32, k=4,
                      dtype=DTYPE_BF16, act=ACT_GELU_ERF, seed=1235),
    "medium": Workload("medium", T=16384, d=2048, r=256, h=1024, E=64, k=8,
                       dtype=DTYPE_BF16, act=ACT_GELU_ERF, seed=1236, gate_bias="zipf"),
    "large": Workload("large", T=32768, d=4096, r=512, h=2048, E=128, k=8,
                      dtype=DTYPE_BF16, act=ACT_GELU_ERF, seed=1237),
    "decode": Workload("decode", T=512, d=2048, r=256, h=1024, E=64, k=8,
                       dtype=DTYPE_BF16, act=ACT_GELU_ERF, seed=1238),
}
DECODE_TOKEN_COUNTS = (1, 8, 64, 512)

_TAGS = {"x": 1, "dy": 2, "w_gate": 3, "w_down": 4, "w1": 5, "w2": 6, "w_up": 7, "b1": 8, "b2": 9}


def _round_chunk_inplace(bits: np.ndarray) -> None:
    step = 1 << 20                                  # cache-sized pieces, no full-size temporaries
    for i in range(0, bits.size, step):
        b = bits[i:i + step]
        lsb = (b >> np.uint32(16)) & np.uint32(1)
        b += np.uint32(0x7FFF)
        b += lsb
        b &= np.uint32(0xFFFF0000)


def bf16_round(a: np.ndarray, inplace: bool = False) -> np.ndarray:
    """Round float32 values to the nearest bf16 value (ties to even); result stays float32."""
    out = a if inplace and a.dtype == np.float32 and a.flags.c_contiguous else np.array(a, dtype=np.float32, order="C", copy=True)
    flat = out.reshape(-1).view(np.uint32)
    if flat.size < (1 << 22):
        _round_chunk_inplace(flat)
    else:                                           # numpy releases the GIL inside ufuncs
        from concurrent.futures import ThreadPoolExecutor
        n = min(16, os.cpu_count() or 1)
        bounds = np.linspace(0, flat.size, n + 1).astype(np.int64)
        with ThreadPoolExecutor(n) as pool:
            list(pool.map(lambda i: _round_chunk_inplace(flat[bounds[i]:bounds[i + 1]]), range(n)))
    return out


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal(seed: int, tag: int, attempt: int, shape, std: float, dtype: int) -> np.ndarray:
    gen = np.random.Generator(np.random.Philox(key=[(seed << 16) ^ tag, attempt]))
    a = gen.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return bf16_round(a, inplace=True) if dtype == DTYPE_BF16 else a


def zipf_log_popularity(E: int, s: float = 1.1) -> np.ndarray:
    """ln q_e with q_e proportional to (e+1)^-s, normalised over the E experts."""
    q = (np.arange(E, dtype=np.float64) + 1.0) ** (-s)
    q /= q.sum()
    return np.log(q).astype(np.float32)


def make_inputs(w: Workload, with_dy: bool = True) -> Dict[str, Optional[np.ndarray]]:
    """Draw every tensor of one layer call.

    x, dy ~ N(0,1); weights ~ N(0, fan_in^-1/2), stored [out_features, in_features]:
    w_gate [E,d] ([E,r] when the gate reads x'), w_down [r,d], w1 [E,h,r], w2 [E,r,h], w_up [d,r].  b_gate is fp32 [E] or None.
    The projection-free layer (cdac) has r == d and no w_down / w_up (None).
    """
    s, dt = w.seed, w.dtype
    out: Dict[str, Optional[np.ndarray]] = {
        "x": _normal(s, _TAGS["x"], 0, (w.T, w.d), 1.0, dt),
        "w_gate": (_normal(s, _TAGS["w_gate"], 0, (w.E, w.r), w.r ** -0.5, dt) if w.gate_low
                   else _normal(s, _TAGS["w_gate"], 0, (w.E, w.d), w.d ** -0.5, dt)),
        "w_down": None if w.cdac else _normal(s, _TAGS["w_down"], 0, (w.r, w.d), w.d ** -0.5, dt),
        "w1": _normal(s, _TAGS["w1"], 0, (w.E, w.h, w.r), w.r ** -0.5, dt),
        "w2": _normal(s, _TAGS["w2"], 0, (w.E, w.r, w.h), w.h ** -0.5, dt),
        "w_up": None if w.cdac else _normal(s, _TAGS["w_up"], 0, (w.d, w.r), w.r ** -0.5, dt),
        "b_gate": zipf_log_popularity(w.E) if w.gate_bias == "zipf" else None,
        "dy": _normal(s, _TAGS["dy"], 0, (w.T, w.d), 1.0, dt) if with_dy else None,
    }
    if w.expert_bias:                                # fp32 whatever the workload dtype, like the gate bias
        out["b1"] = _normal(s, _TAGS["b1"], 0, (w.E, w.h), 0.5, DTYPE_F32)
        out["b2"] = _normal(s, _TAGS["b2"], 0, (w.E, w.r), 0.5, DTYPE_F32)
    return out


def redraw_rows(w: Workload, x: np.ndarray, rows: np.ndarray, attempt: int) -> None:
    """Replace the given token rows of x, in place, by fresh draws of stream `attempt` (>= 1)."""
    rows = np.asarray(rows, dtype=np.int64)
    if rows.size == 0:
        return
    x[rows] = _normal(w.seed, _TAGS["x"], attempt, (rows.size, w.d), 1.0, w.dtype)
