"""Pins of the oracle's gate-on-x' variant (the alternative the text after Eq. 2 mentions: the gate reads the
low-width token, w_gate is [E,r]) to things other than the oracle.  CPU only."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
from oracle import margin
from paper_2502_16927_b200 import workloads as wl

from helpers import small_workload, regrid


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def _low_gate(w, inp, seed=5, grid=2.0 ** -10):
    g = np.random.default_rng(seed)
    inp["w_gate"] = (np.round(g.standard_normal((w.E, w.r)) * w.r ** -0.5 / grid) * grid).astype(np.float32)
    return inp


def test_logits_are_two_library_matmuls_and_rounding_is_to_bf16():
    w, inp = small_workload(T=19, d=11, r=6, h=5, E=7, k=2, bias=True)
    _low_gate(w, inp)
    x_lo = _f64(inp["x"]) @ _f64(inp["w_down"]).T
    ref = x_lo @ _f64(inp["w_gate"]).T + _f64(inp["b_gate"])
    np.testing.assert_allclose(oracle.gate_logits_low(inp["x"], inp["w_down"], inp["w_gate"], inp["b_gate"]), ref, rtol=0, atol=1e-13)
    x_lo_r = _f64(wl.bf16_round(x_lo.astype(np.float32)))          # fp64 -> fp32 is exact enough here: grid values
    ref_r = x_lo_r @ _f64(inp["w_gate"]).T + _f64(inp["b_gate"])
    got_r = oracle.gate_logits_low(inp["x"], inp["w_down"], inp["w_gate"], inp["b_gate"], round_x_lo_bf16=True)
    np.testing.assert_allclose(got_r, ref_r, rtol=0, atol=1e-13)
    assert np.abs(got_r - ref).max() > 1e-6                          # the rounding is really applied


def test_with_an_identity_descend_projection_both_gates_are_the_same_layer():
    w, inp = small_workload(T=16, d=8, r=8, h=6, E=4, k=2, bias=True)
    inp["w_down"] = np.eye(8, dtype=np.float32)
    rt_x = oracle.route(inp, w.k)
    rt_lo = oracle.route(inp, w.k, gate_low=True)                    # w_gate [E, d] = [E, r]
    np.testing.assert_array_equal(rt_x.topk_idx, rt_lo.topk_idx)
    np.testing.assert_allclose(rt_x.logits, rt_lo.logits, rtol=0, atol=1e-13)
    a, b = oracle.backward_full(inp, rt_x, w.act), oracle.backward_full(inp, rt_lo, w.act)
    for key in ("y", "dx", "dw_gate", "db_gate", "dw_up"):
        np.testing.assert_allclose(a[key], b[key], rtol=0, atol=1e-12)
    # dW_down: with gate on x the gate's share goes to dx directly; with gate on x' it passes through W_down = I
    gate_share = (_dense(rt_x, a["dlogit"]) @ _f64(inp["w_gate"])).T @ _f64(inp["x"])      # [r, d]
    np.testing.assert_allclose(b["dw_down"] - a["dw_down"], gate_share, rtol=0, atol=1e-12)


def _dense(rt, dl):
    out = np.zeros(rt.logits.shape)
    np.put_along_axis(out, rt.topk_idx.astype(np.int64), dl, axis=1)
    return out


def _conditioned(**kw):
    w, inp = small_workload(act=wl.ACT_GELU_ERF, bias=True, **kw)
    _low_gate(w, inp)
    for _ in range(8):
        margin.enforce_margin(w, inp, margin=0.08, gate_low=True)
        regrid(w, inp)
        if margin.min_topk_gap(oracle.gate_logits_low(inp["x"], inp["w_down"], inp["w_gate"], inp["b_gate"]), w.k).min() >= 0.07:
            return w, inp
    raise AssertionError("could not condition the workload")


def _loss(inp, w):
    rt = oracle.route(inp, w.k, gate_low=True)
    return float(np.sum(oracle.forward_tokens(inp, rt, w.act)["y"] * _f64(inp["dy"]))), rt


def test_gradients_with_the_gate_on_the_low_width_token_match_finite_differences():
    w, inp = _conditioned(T=10, d=9, r=5, h=7, E=4, k=2)
    _, rt = _loss(inp, w)
    grads = oracle.backward_full(inp, rt, w.act)
    analytic = {"x": grads["dx"], "w_gate": grads["dw_gate"], "b_gate": grads["db_gate"],
                "w_down": grads["dw_down"], "w_up": grads["dw_up"],
                "w1": np.stack([grads["dw1"][e] for e in range(w.E)]),
                "w2": np.stack([grads["dw2"][e] for e in range(w.E)])}
    assert analytic["w_gate"].shape == (w.E, w.r)
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
                val, rt_p = _loss(dict(inp, **{key: pert}), w)
                np.testing.assert_array_equal(rt_p.topk_idx, rt.topk_idx)
                vals.append(val)
            fd = (-vals[0] + 8 * vals[1] - 8 * vals[2] + vals[3]) / (12 * delta)
            assert abs(fd - an[index]) <= 2e-7 * max(abs(an[index]), scale), (key, index, fd, an[index])
