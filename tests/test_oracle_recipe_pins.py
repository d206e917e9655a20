"""Pins of the oracle's training-recipe variants (Table 5: capacity factor, load-balancing loss) to things
other than the oracle: hand-computed capacities, a brute-force per-expert list, a numpy re-statement of the
dropped forward, closed forms of the loss and central finite differences.  CPU only."""
from __future__ import annotations

import numpy as np
import pytest
from scipy.special import erf, softmax

import oracle
from oracle import margin
from paper_2502_16927_b200 import workloads as wl

from helpers import small_workload, regrid


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def _gelu(z):
    return 0.5 * z * (1.0 + erf(z / np.sqrt(2.0)))


# ---------------------------------------------------------------- capacity: the tables

def test_capacity_rows_of_hand_computed_cases():
    assert oracle.capacity_rows(160, 8, 128, 1.2) == 12          # 1.2 * 10 rows, exactly
    assert oracle.capacity_rows(100, 2, 8, 1.0) == 25
    assert oracle.capacity_rows(10, 2, 8, 1.25) == 4             # ceil(3.125)
    assert oracle.capacity_rows(7, 1, 4, 1.0) == 2               # ceil(1.75)
    assert oracle.capacity_rows(32768, 8, 128, 1.2) == 2458      # Table 5's factor at the benchmark shape: ceil(2457.6)


@pytest.mark.parametrize("T,E,k,cap", [(40, 4, 2, 13), (64, 8, 3, 5), (9, 5, 5, 1), (33, 3, 1, 40), (50, 6, 2, 0)])
def test_capacity_tables_match_a_brute_force_list_per_expert(T, E, k, cap):
    g = np.random.default_rng(T + E)
    # skewed choices so that some experts overflow and some do not; the k choices of a token are distinct
    idx = np.stack([g.choice(E, size=k, replace=False, p=np.arange(1, E + 1) / (E * (E + 1) / 2)) for _ in range(T)])
    chosen, counts, offsets, ros, sor, keep = oracle.tables_capacity(idx.astype(np.int32), E, cap)
    flat = idx.ravel()
    lists = [[s for s in range(T * k) if flat[s] == e] for e in range(E)]         # ascending slot id
    exp_rows, exp_keep, row = {}, np.zeros(T * k, dtype=np.uint8), 0
    for e in range(E):
        assert chosen[e] == len(lists[e])
        assert counts[e] == min(len(lists[e]), cap)
        assert offsets[e] == row
        for s in lists[e][:cap]:
            exp_rows[s] = row
            exp_keep[s] = 1
            row += 1
    assert offsets[E] == row
    np.testing.assert_array_equal(keep, exp_keep)
    for s in range(T * k):
        assert ros[s] == exp_rows.get(s, -1)
    for r_ in range(T * k):
        assert sor[r_] == ([s for s, rr in exp_rows.items() if rr == r_] or [-1])[0]


def test_a_capacity_nobody_reaches_gives_the_dropless_tables():
    g = np.random.default_rng(1)
    idx = np.stack([g.choice(7, size=3, replace=False) for _ in range(50)]).astype(np.int32)
    chosen, counts, offsets, ros, sor, keep = oracle.tables_capacity(idx, 7, 10 ** 6)
    c0, o0, r0, s0 = oracle.tables(idx, 7)
    for a, b in ((counts, c0), (chosen, c0), (offsets, o0), (ros, r0), (sor, s0)):
        np.testing.assert_array_equal(a, b)
    assert keep.all()


# ---------------------------------------------------------------- capacity: the forward

def test_single_expert_with_capacity_is_an_mlp_on_the_first_rows_and_zero_after():
    w, inp = small_workload(T=21, d=10, r=6, h=14, E=1, k=1, act=wl.ACT_GELU_ERF)
    f = 0.5
    cap = oracle.capacity_rows(21, 1, 1, f)
    assert cap == 11
    rt = oracle.route(inp, 1, capacity_factor=f)
    x_lo = _f64(inp["x"]) @ _f64(inp["w_down"]).T
    mlp = (_gelu(x_lo @ _f64(inp["w1"][0]).T) @ _f64(inp["w2"][0]).T) @ _f64(inp["w_up"]).T
    mlp[cap:] = 0.0
    np.testing.assert_allclose(oracle.forward_tokens(inp, rt, w.act)["y"], mlp, rtol=0, atol=1e-12)
    np.testing.assert_allclose(oracle.forward_grouped(inp, rt, w.act)["y"], mlp, rtol=0, atol=1e-12)


def test_dropped_forward_against_a_numpy_restatement():
    """y[t] = (sum over kept slots of p_j sigma(x' W1_e^T) W2_e^T) W_up^T, p = softmax over the k chosen logits of
    ALL k slots (dropping does not renormalise), written with library matmuls, a library softmax and the
    brute-force keep rule."""
    w, inp = small_workload(T=40, d=12, r=6, h=10, E=5, k=3, act=wl.ACT_GELU_ERF, bias=True)
    inp["b_gate"] = (inp["b_gate"] + np.float32(0.5) * np.arange(5, dtype=np.float32)).astype(np.float32)   # skew
    f = 0.8
    rt = oracle.route(inp, w.k, capacity_factor=f)
    cap = int(np.ceil(f * 40 * 3 / 5))
    assert rt.keep.sum() < rt.keep.size and rt.keep.sum() > 0
    logits = _f64(inp["x"]) @ _f64(inp["w_gate"]).T + _f64(inp["b_gate"])
    order = np.argsort(-logits, axis=1, kind="stable")[:, :w.k]
    p = softmax(np.take_along_axis(logits, order, axis=1), axis=1)
    seen = np.zeros(w.E, dtype=int)
    x_lo = _f64(inp["x"]) @ _f64(inp["w_down"]).T
    y = np.zeros((w.T, w.d))
    for t in range(w.T):
        y_lo = np.zeros(w.r)
        for j in range(w.k):
            e = order[t, j]
            kept = seen[e] < cap
            seen[e] += 1
            if kept:
                y_lo += p[t, j] * (_gelu(x_lo[t] @ _f64(inp["w1"][e]).T) @ _f64(inp["w2"][e]).T)
        y[t] = y_lo @ _f64(inp["w_up"]).T
    np.testing.assert_allclose(oracle.forward_tokens(inp, rt, w.act)["y"], y, rtol=0, atol=1e-12)
    np.testing.assert_allclose(oracle.forward_grouped(inp, rt, w.act)["y"], y, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- load-balancing loss: closed forms

def test_aux_loss_closed_forms():
    T, E, k, alpha = 24, 6, 2, 0.001
    g = np.random.default_rng(0)
    idx = np.stack([g.choice(E, size=k, replace=False) for _ in range(T)]).astype(np.int32)
    # equal logits: P_e = 1/E whatever the routing, and the f_e sum to 1  ->  L = alpha
    loss, grad = oracle.aux_loss(np.zeros((T, E)), idx, alpha)
    assert abs(loss - alpha) < 1e-15
    # ... and the gradient is (alpha E / T)(1/E)(f_e - 1/E)
    f = np.bincount(idx.ravel(), minlength=E) / (T * k)
    np.testing.assert_allclose(grad, np.tile(alpha / T * (f - 1.0 / E), (T, 1)), rtol=0, atol=1e-18)
    # collapse: every token puts (almost) all probability on expert 0 and k = 1 routes there  ->  L = alpha E
    logits = np.zeros((T, E)); logits[:, 0] = 60.0
    loss, _ = oracle.aux_loss(logits, np.zeros((T, 1), dtype=np.int32), alpha)
    assert abs(loss - alpha * E) < 1e-15
    # perfectly balanced and confident, k = 1: token t -> expert t mod E  ->  L = alpha E * E * (1/E)(1/E) = alpha
    logits = np.zeros((T, E)); logits[np.arange(T), np.arange(T) % E] = 60.0
    loss, _ = oracle.aux_loss(logits, (np.arange(T) % E).astype(np.int32)[:, None], alpha)
    assert abs(loss - alpha) < 1e-15
    # a hand-computed two-expert case: T = 2, k = 1, logits (ln 3, 0) and (0, 0), both routed to expert 0:
    # p = (3/4, 1/4), (1/2, 1/2); P = (5/8, 3/8); f = (1, 0); L = alpha * 2 * 5/8
    loss, _ = oracle.aux_loss(np.array([[np.log(3.0), 0.0], [0.0, 0.0]]), np.zeros((2, 1), dtype=np.int32), 0.5)
    assert abs(loss - 0.5 * 2 * 5 / 8) < 1e-15


def test_aux_loss_gradient_matches_finite_differences_and_rows_sum_to_zero():
    T, E, k, alpha = 9, 5, 2, 0.37
    g = np.random.default_rng(4)
    logits = g.standard_normal((T, E))
    idx, _ = oracle.topk(logits, k)
    _, grad = oracle.aux_loss(logits, idx, alpha)
    np.testing.assert_allclose(grad.sum(axis=1), 0.0, atol=1e-17)
    delta = 1e-4
    for t in range(T):
        for e in range(E):
            vals = []
            for mult in (2, 1, -1, -2):
                pert = logits.copy(); pert[t, e] += mult * delta
                vals.append(oracle.aux_loss(pert, idx, alpha, want_grad=False)[0])      # routing (f) held fixed
            fd = (-vals[0] + 8 * vals[1] - 8 * vals[2] + vals[3]) / (12 * delta)
            assert abs(fd - grad[t, e]) <= 1e-9 * np.abs(grad).max(), (t, e, fd, grad[t, e])


# ---------------------------------------------------------------- gradients of the whole layer under both settings

def _conditioned(**kw):
    w, inp = small_workload(act=wl.ACT_GELU_ERF, bias=True, **kw)
    inp["b_gate"] = (inp["b_gate"] + np.float32(0.25) * np.arange(w.E, dtype=np.float32)).astype(np.float32)
    for _ in range(8):
        margin.enforce_margin(w, inp, margin=0.08)
        regrid(w, inp)
        if margin.min_topk_gap(oracle.gate_logits(inp["x"], inp["w_gate"], inp["b_gate"]), w.k).min() >= 0.07:
            return w, inp
    raise AssertionError("could not condition the workload")


def _loss(inp, w, f, alpha):
    rt = oracle.route(inp, w.k, capacity_factor=f)
    val = float(np.sum(oracle.forward_tokens(inp, rt, w.act)["y"] * _f64(inp["dy"])))
    if alpha > 0:
        val += oracle.aux_loss(rt.logits, rt.topk_idx, alpha, want_grad=False)[0]
    return val, rt


@pytest.mark.parametrize("f,alpha", [(0.75, 0.0), (0.0, 0.3), (0.75, 0.3)])
def test_gradients_with_capacity_and_aux_loss_match_finite_differences(f, alpha):
    w, inp = _conditioned(T=12, d=9, r=5, h=7, E=4, k=2)
    _, rt = _loss(inp, w, f, alpha)
    if f > 0:
        assert 0 < rt.keep.sum() < rt.keep.size                     # something is dropped, something is kept
    grads = oracle.backward_full(inp, rt, w.act, aux_alpha=alpha)
    analytic = {"x": grads["dx"], "w_gate": grads["dw_gate"], "b_gate": grads["db_gate"],
                "w_down": grads["dw_down"], "w_up": grads["dw_up"],
                "w1": np.stack([grads["dw1"][e] for e in range(w.E)]),
                "w2": np.stack([grads["dw2"][e] for e in range(w.E)])}
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
                val, rt_p = _loss(dict(inp, **{key: pert}), w, f, alpha)
                np.testing.assert_array_equal(rt_p.topk_idx, rt.topk_idx)           # routing did not move
                vals.append(val)
            fd = (-vals[0] + 8 * vals[1] - 8 * vals[2] + vals[3]) / (12 * delta)
            assert abs(fd - an[index]) <= 2e-7 * max(abs(an[index]), scale), (key, index, fd, an[index])


def test_a_token_with_every_slot_dropped_gets_no_gradient_from_the_experts():
    w, inp = _conditioned(T=12, d=9, r=5, h=7, E=4, k=2)
    rt = oracle.route(inp, w.k, capacity_factor=0.5)
    all_dropped = np.where(rt.keep.reshape(w.T, w.k).sum(axis=1) == 0)[0]
    assert all_dropped.size > 0
    bwd = oracle.backward_tokens(inp, rt, w.act)
    fwd = oracle.forward_tokens(inp, rt, w.act)
    assert np.all(fwd["y"][all_dropped] == 0.0)
    assert np.all(bwd["dx"][all_dropped] == 0.0) and np.all(bwd["dlogit"][all_dropped] == 0.0)
