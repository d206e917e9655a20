"""Pins of the oracle's expert-bias variant (z = x' W1^T + b1, u = sigma(z) W2^T + b2; Eq. 4 itself has no biases)
to things other than the oracle.  CPU only."""
from __future__ import annotations

import numpy as np
import pytest
from scipy.special import erf

import oracle
from oracle import margin
from paper_2502_16927_b200 import workloads as wl

from helpers import small_workload, regrid


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def _with_biases(w, inp, seed=11, grid=2.0 ** -10):
    g = np.random.default_rng(seed)
    inp["b1"] = (np.round(g.standard_normal((w.E, w.h)) * 0.5 / grid) * grid).astype(np.float32)
    inp["b2"] = (np.round(g.standard_normal((w.E, w.r)) * 0.5 / grid) * grid).astype(np.float32)
    return inp


def test_single_expert_with_biases_is_an_mlp_with_biases():
    w, inp = small_workload(T=21, d=10, r=6, h=14, E=1, k=1, act=wl.ACT_GELU_ERF)
    _with_biases(w, inp)
    rt = oracle.route(inp, 1)
    x_lo = _f64(inp["x"]) @ _f64(inp["w_down"]).T
    z = x_lo @ _f64(inp["w1"][0]).T + _f64(inp["b1"][0])
    a = 0.5 * z * (1.0 + erf(z / np.sqrt(2.0)))
    ref = (a @ _f64(inp["w2"][0]).T + _f64(inp["b2"][0])) @ _f64(inp["w_up"]).T
    np.testing.assert_allclose(oracle.forward_tokens(inp, rt, w.act)["y"], ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(oracle.forward_grouped(inp, rt, w.act)["y"], ref, rtol=0, atol=1e-12)


def test_zero_biases_change_nothing_and_b2_alone_adds_the_gate_weighted_bias():
    w, inp = small_workload(T=30, d=12, r=6, h=10, E=5, k=2, act=wl.ACT_GELU_TANH, bias=True)
    rt = oracle.route(inp, w.k)
    base = oracle.backward_full(inp, rt, w.act)
    zero = dict(inp, b1=np.zeros((w.E, w.h), np.float32), b2=np.zeros((w.E, w.r), np.float32))
    got = oracle.backward_full(zero, rt, w.act)
    for key in ("y", "dx", "dw_gate", "dw_up", "dw_down"):
        np.testing.assert_array_equal(got[key], base[key])
    # b2 only: y' gains sum_j p_j b2[e_j], a closed form in the routing tables
    b2 = np.random.default_rng(2).standard_normal((w.E, w.r)).astype(np.float32)
    only_b2 = dict(zero, b2=b2)
    extra = np.einsum("tj,tjc->tc", rt.topk_p, _f64(b2)[rt.topk_idx]) @ _f64(inp["w_up"]).T
    np.testing.assert_allclose(oracle.forward_tokens(only_b2, rt, w.act)["y"], base["y"] + extra, rtol=0, atol=1e-12)


def _conditioned(**kw):
    w, inp = small_workload(act=wl.ACT_GELU_ERF, bias=True, **kw)
    _with_biases(w, inp)
    for _ in range(8):
        margin.enforce_margin(w, inp, margin=0.08)
        regrid(w, inp)
        if margin.min_topk_gap(oracle.gate_logits(inp["x"], inp["w_gate"], inp["b_gate"]), w.k).min() >= 0.07:
            return w, inp
    raise AssertionError("could not condition the workload")


def _loss(inp, w):
    rt = oracle.route(inp, w.k)
    return float(np.sum(oracle.forward_tokens(inp, rt, w.act)["y"] * _f64(inp["dy"]))), rt


def test_gradients_with_expert_biases_match_finite_differences():
    w, inp = _conditioned(T=10, d=9, r=5, h=7, E=4, k=2)
    _, rt = _loss(inp, w)
    grads = oracle.backward_full(inp, rt, w.act)
    analytic = {"x": grads["dx"], "w_gate": grads["dw_gate"], "b_gate": grads["db_gate"], "b1": grads["db1"], "b2": grads["db2"],
                "w_down": grads["dw_down"], "w_up": grads["dw_up"],
                "w1": np.stack([grads["dw1"][e] for e in range(w.E)]),
                "w2": np.stack([grads["dw2"][e] for e in range(w.E)])}
    per_expert = oracle.backward_full(inp, rt, w.act, experts=[1, 3])
    for e in (1, 3):                                   # the per-expert entry point agrees with the all-experts one
        np.testing.assert_array_equal(per_expert["db1"][e], grads["db1"][e])
        np.testing.assert_array_equal(per_expert["dw2"][e], grads["dw2"][e])
    g = np.random.default_rng(3)
    delta = 2.0 ** -8
    for key, an in analytic.items():
        scale = np.sqrt(np.mean(an ** 2))
        assert scale > 0
        for flat in g.choice(an.size, size=min(an.size, 12), replace=False):
            index = np.unravel_index(flat, an.shape)
            vals = []
            for mult in (2, 1, -1, -2):
                pert = inp[key].copy()
                pert[index] = np.float32(inp[key][index] + mult * delta)
                assert float(pert[index]) == float(inp[key][index]) + mult * delta
                vals.append(_loss(dict(inp, **{key: pert}), w)[0])
            fd = (-vals[0] + 8 * vals[1] - 8 * vals[2] + vals[3]) / (12 * delta)
            assert abs(fd - an[index]) <= 2e-7 * max(abs(an[index]), scale), (key, index, fd, an[index])
