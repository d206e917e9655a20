"""Closed-form counts from the paper's Table 3 (parameters, FLOPs per iteration, All-to-All bytes)
for a GPT-style model whose FFNs are fine-grained or BigMac MoE layers.  TEST INFRASTRUCTURE ONLY.

Symbols are the paper's (Table 2): b*s tokens per iteration, h hidden width, l layers, v vocabulary,
e experts, top_k, r downscaling ratio, ep expert-parallel degree.  The All-to-All figure is bytes at
2 bytes per element (the factor 8 = 2 All-to-Alls x forward+backward x 2 bytes).
"""
from __future__ import annotations


def params(h, l, v, e, r, bigmac: bool) -> float:
    base = (4 * h * h + 8 * h + (2 * r * h * h + 2 * r * h) * e) * l + (v + e + 2) * h
    return base + (2 * r * l * h * h if bigmac else 0)


def flops(bs, s, h, l, v, r, top_k, bigmac: bool) -> float:
    base = 12 * bs * l * h * h * (2 + s / h + v / (2 * l * h) + r * top_k)
    return base + (12 * r * bs * l * h * h if bigmac else 0)


def a2a_bytes(bs, h, l, top_k, ep, r, bigmac: bool) -> float:
    base = 8 * bs * l * h * top_k * (ep - 1) / ep
    return base * (r if bigmac else 1)


def layer_a2a_elements(bs, h, top_k, ep, r=1.0) -> float:
    """Eq. 1: elements crossing the two All-to-Alls of one MoE layer in one pass; r scales the row width."""
    return 2 * top_k * (ep - 1) / ep * bs * h * r
