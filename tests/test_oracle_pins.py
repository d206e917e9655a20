"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without any GPU.

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong sign or
index, a transposed operand) fails at least one of them.
"""
import os

import numpy as np
import pytest
from scipy.special import erf, softmax

import oracle
from oracle import counts, margin
from paper_2502_16927_b200 import workloads as wl

from helpers import small_workload, regrid

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _act(act, z):
    if act == wl.ACT_RELU:
        return np.maximum(z, 0.0)
    if act == wl.ACT_GELU_ERF:
        return 0.5 * z * (1.0 + erf(z / np.sqrt(2.0)))
    if act == wl.ACT_GELU_TANH:
        return 0.5 * z * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (z + 0.044715 * z ** 3)))
    return z


def _f64(a):
    return np.asarray(a, dtype=np.float64)


# ---------------------------------------------------------------- routing: top-k and gate weights

def test_gate_logits_match_library_matmul():
    w, inp = small_workload(T=37, d=19, E=5, bias=True)
    ref = _f64(inp["x"]) @ _f64(inp["w_gate"]).T + _f64(inp["b_gate"])
    np.testing.assert_allclose(oracle.gate_logits(inp["x"], inp["w_gate"], inp["b_gate"]), ref, rtol=0, atol=1e-13)
    ref0 = _f64(inp["x"]) @ _f64(inp["w_gate"]).T
    np.testing.assert_allclose(oracle.gate_logits(inp["x"], inp["w_gate"]), ref0, rtol=0, atol=1e-13)


@pytest.mark.parametrize("E,k", [(8, 2), (8, 8), (1, 1), (5, 1), (7, 3)])
def test_topk_is_the_full_sort(E, k):
    g = np.random.default_rng(E * 10 + k)
    logits = g.standard_normal((50, E))
    idx, p = oracle.topk(logits, k)
    order = np.argsort(-logits, axis=1, kind="stable")[:, :k]
    np.testing.assert_array_equal(idx, order.astype(np.int32))
    for t in range(logits.shape[0]):
        assert len(set(idx[t])) == k                       # k distinct experts per token
        sel = logits[t, idx[t]]
        assert np.all(np.diff(sel) <= 0)                   # slot order = descending logit
        rest = np.delete(logits[t], idx[t])
        assert rest.size == 0 or rest.max() <= sel.min()   # nothing unselected beats a selected one
    np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=0, atol=1e-12)
    np.testing.assert_allclose(p, softmax(np.take_along_axis(logits, order, 1), axis=1), rtol=0, atol=1e-14)
    if k == 1:
        np.testing.assert_array_equal(p, np.ones_like(p))


def test_topk_ties_go_to_the_lower_expert_and_equal_logits_share_equally():
    logits = np.array([[0.5, 2.0, 2.0, -1.0, 2.0], [1.0, 1.0, 1.0, 1.0, 1.0]])
    idx, p = oracle.topk(logits, 2)
    np.testing.assert_array_equal(idx, [[1, 2], [0, 1]])
    np.testing.assert_allclose(p, 0.5, rtol=0, atol=1e-15)
    idx, p = oracle.topk(logits, 5)
    np.testing.assert_array_equal(idx[1], [0, 1, 2, 3, 4])
    np.testing.assert_allclose(p[1], 0.2, rtol=0, atol=1e-15)


# ---------------------------------------------------------------- histogram, offsets, permutation

@pytest.mark.parametrize("T,E,k", [(40, 8, 2), (1, 8, 3), (33, 1, 1), (17, 6, 6), (64, 16, 1)])
def test_tables_are_a_stable_counting_sort(T, E, k):
    g = np.random.default_rng(T + E + k)
    idx = np.stack([g.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    counts_, offsets, ros, sor = oracle.tables(idx, E)
    N = T * k
    flat = idx.ravel()
    np.testing.assert_array_equal(counts_, np.bincount(flat, minlength=E))
    assert counts_.sum() == N                                              # dropless
    np.testing.assert_array_equal(offsets, np.concatenate([[0], np.cumsum(counts_)]))
    np.testing.assert_array_equal(np.sort(ros), np.arange(N))             # bijection
    np.testing.assert_array_equal(sor[ros], np.arange(N))                 # inverse
    np.testing.assert_array_equal(sor, np.argsort(flat, kind="stable"))   # library routine
    for e in range(E):
        seg = sor[offsets[e]:offsets[e + 1]]
        assert np.all(flat[seg] == e) and np.all(np.diff(seg) > 0)        # ascending slot id
    for s in range(N):                                                     # brute force definition
        assert ros[s] == offsets[flat[s]] + int(np.sum(flat[:s] == flat[s]))


# ---------------------------------------------------------------- dispatch / combine

def test_dispatch_is_a_pure_copy_and_unit_weight_combine_sums_k_copies():
    w, inp = small_workload(T=29, E=6, k=3, act=wl.ACT_IDENTITY, r=8, h=8)
    eye = np.eye(8, dtype=np.float32)
    inp["w1"] = np.tile(eye, (6, 1, 1))
    inp["w2"] = np.tile(eye, (6, 1, 1))
    rt = oracle.route(inp, w.k)
    x_lo = _f64(inp["x"]) @ _f64(inp["w_down"]).T
    grouped = oracle.forward_grouped(inp, rt, w.act)
    x_lo_oracle = oracle.forward_tokens(inp, rt, w.act)["x_lo"]
    np.testing.assert_allclose(x_lo_oracle, x_lo, rtol=0, atol=1e-13)
    for s in range(w.N):                                                   # bitwise: dispatch only copies
        np.testing.assert_array_equal(grouped["xg"][rt.row_of_slot[s]], x_lo_oracle[s // w.k])
    np.testing.assert_allclose(grouped["y_lo"], x_lo, rtol=0, atol=1e-13)   # sum_j p_j x' = x'
    ones = oracle.Routing(rt.logits, rt.topk_idx, np.ones_like(rt.topk_p), rt.counts, rt.offsets,
                          rt.row_of_slot, rt.slot_of_row)
    np.testing.assert_allclose(oracle.forward_grouped(inp, ones, w.act)["y_lo"], w.k * x_lo, rtol=0, atol=1e-13)
    np.testing.assert_allclose(oracle.forward_tokens(inp, ones, w.act)["y_lo"], w.k * x_lo, rtol=0, atol=1e-13)
    # identity experts: the layer collapses to the two shared projections (Eq. 2 with E_i = id)
    y_ref = x_lo @ _f64(inp["w_up"]).T
    np.testing.assert_allclose(oracle.forward_tokens(inp, rt, w.act)["y"], y_ref, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- expert FFN and projections

def _mlp(inp, e, act):
    x_lo = _f64(inp["x"]) @ _f64(inp["w_down"]).T
    a = _act(act, x_lo @ _f64(inp["w1"][e]).T)
    return (a @ _f64(inp["w2"][e]).T) @ _f64(inp["w_up"]).T


@pytest.mark.parametrize("act", [wl.ACT_RELU, wl.ACT_GELU_ERF, wl.ACT_GELU_TANH, wl.ACT_IDENTITY])
def test_single_expert_is_a_four_matmul_mlp(act):
    w, inp = small_workload(T=21, d=10, r=6, h=14, E=1, k=1, act=act)
    rt = oracle.route(inp, 1)
    np.testing.assert_allclose(oracle.forward_tokens(inp, rt, act)["y"], _mlp(inp, 0, act), rtol=0, atol=1e-12)
    np.testing.assert_allclose(oracle.forward_grouped(inp, rt, act)["y"], _mlp(inp, 0, act), rtol=0, atol=1e-12)


def test_identity_projections_give_the_conventional_layer_of_eq3():
    """Eq. 3 (y = sum_{i in T} p_i(x) E_i(x), experts d -> m -> d) written out token by token with numpy, against
    the oracle's Eq. 2 evaluated with W_down = W_up = I: the projection-free layer is that special case, and its
    dx is the sum of the expert path and the gate path."""
    T, d, m, E, k = 19, 8, 5, 6, 3
    w = wl.Workload("cdac", T=T, d=d, r=d, h=m, E=E, k=k, dtype=wl.DTYPE_F32, act=wl.ACT_GELU_ERF, seed=41, cdac=True)
    inp = wl.make_inputs(w)
    assert inp["w_down"] is None and inp["w_up"] is None and inp["w1"].shape == (E, m, d) and inp["w2"].shape == (E, d, m)
    x, wg, w1, w2 = (_f64(inp[key]) for key in ("x", "w_gate", "w1", "w2"))
    y = np.zeros((T, d))
    for t in range(T):
        logits = wg @ x[t]
        chosen = sorted(range(E), key=lambda e: (-logits[e], e))[:k]
        p = softmax(logits[chosen])
        for p_i, e in zip(p, chosen):
            y[t] += p_i * (w2[e] @ _act(w.act, w1[e] @ x[t]))
    full = dict(inp, w_down=np.eye(d, dtype=np.float32), w_up=np.eye(d, dtype=np.float32))
    rt = oracle.route(full, k)
    np.testing.assert_allclose(oracle.forward_tokens(full, rt, w.act)["y"], y, rtol=0, atol=1e-12)
    # parameter parity of the twin: experts of d -> r -> h -> r -> d and d -> m -> d hold the same number of weights
    big = wl.WORKLOADS["large"]
    twin = big.cdac_twin()
    assert (twin.r, twin.h) == (4096, 256) and 2 * twin.r * twin.h == 2 * big.r * big.h


def test_identical_experts_make_the_output_independent_of_routing():
    w, inp = small_workload(T=31, E=5, k=3, act=wl.ACT_GELU_ERF)
    inp["w1"] = np.tile(inp["w1"][:1], (5, 1, 1))
    inp["w2"] = np.tile(inp["w2"][:1], (5, 1, 1))
    rt = oracle.route(inp, w.k)
    np.testing.assert_allclose(oracle.forward_tokens(inp, rt, w.act)["y"], _mlp(inp, 0, w.act), rtol=0, atol=1e-12)


def test_rectangular_shapes_catch_transposed_operands():
    # all five dimensions distinct: a transposed weight or swapped r/h index cannot go unnoticed
    w, inp = small_workload(T=9, d=11, r=5, h=7, E=3, k=2, act=wl.ACT_GELU_TANH)
    rt = oracle.route(inp, w.k)
    out = oracle.forward_tokens(inp, rt, w.act, want_slots=True)
    x_lo = _f64(inp["x"]) @ _f64(inp["w_down"]).T
    for t in range(w.T):
        y_lo = np.zeros(w.r)
        for j in range(w.k):
            e = rt.topk_idx[t, j]
            z = _f64(inp["w1"][e]) @ x_lo[t]
            u = _f64(inp["w2"][e]) @ _act(w.act, z)
            np.testing.assert_allclose(out["z"][t, j], z, rtol=0, atol=1e-13)
            np.testing.assert_allclose(out["u"][t, j], u, rtol=0, atol=1e-13)
            y_lo += rt.topk_p[t, j] * u
        np.testing.assert_allclose(out["y"][t], _f64(inp["w_up"]) @ y_lo, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- symmetries, two evaluation orders

def test_per_token_and_grouped_evaluation_agree():
    for act in (wl.ACT_RELU, wl.ACT_GELU_ERF):
        w, inp = small_workload(T=45, d=20, r=8, h=24, E=8, k=3, act=act, bias=True)
        rt = oracle.route(inp, w.k)
        a, b = oracle.forward_tokens(inp, rt, act), oracle.forward_grouped(inp, rt, act)
        assert oracle.rel_err(a["y"], b["y"]) < 1e-12 and oracle.rel_err(a["y_lo"], b["y_lo"]) < 1e-12


def test_token_permutation_and_expert_relabelling():
    w, inp = small_workload(T=26, E=6, k=2)
    rt = oracle.route(inp, w.k)
    y = oracle.forward_tokens(inp, rt, w.act)["y"]
    g = np.random.default_rng(0)
    perm = g.permutation(w.T)
    inp_p = dict(inp, x=inp["x"][perm])
    np.testing.assert_array_equal(oracle.forward_tokens(inp_p, oracle.route(inp_p, w.k), w.act)["y"], y[perm])
    ep = g.permutation(w.E)
    inp_e = dict(inp, w_gate=inp["w_gate"][ep], w1=inp["w1"][ep], w2=inp["w2"][ep])
    rt_e = oracle.route(inp_e, w.k)
    np.testing.assert_array_equal(ep[rt_e.topk_idx], rt.topk_idx)
    np.testing.assert_allclose(oracle.forward_tokens(inp_e, rt_e, w.act)["y"], y, rtol=0, atol=1e-13)


def test_subset_evaluation_equals_rows_of_the_full_one():
    w, inp = small_workload(T=30, E=5, k=2)
    rt = oracle.route(inp, w.k)
    tok = np.array([29, 0, 7, 7, 13], dtype=np.int32)
    full_f, full_b = oracle.forward_tokens(inp, rt, w.act), oracle.backward_tokens(inp, rt, w.act)
    np.testing.assert_array_equal(oracle.forward_tokens(inp, rt, w.act, tokens=tok)["y"], full_f["y"][tok])
    np.testing.assert_array_equal(oracle.backward_tokens(inp, rt, w.act, tokens=tok)["dx"], full_b["dx"][tok])


# ---------------------------------------------------------------- gradients

def _loss(inp, w):
    rt = oracle.route(inp, w.k)
    return float(np.sum(oracle.forward_tokens(inp, rt, w.act)["y"] * _f64(inp["dy"]))), rt


def _fd4(inp, w, key, index, delta):
    """4th-order central difference of L = sum(y*dy) w.r.t. one coordinate; all points on the fp32 grid."""
    base = inp[key]
    vals = []
    for mult in (2, 1, -1, -2):
        pert = base.copy()
        pert[index] = np.float32(base[index] + mult * delta)
        assert float(pert[index]) == float(base[index]) + mult * delta
        vals.append(_loss(dict(inp, **{key: pert}), w)[0])
    return (-vals[0] + 8 * vals[1] - 8 * vals[2] + vals[3]) / (12 * delta)


def _conditioned(act, **kw):
    w, inp = small_workload(act=act, bias=True, **kw)
    for _ in range(8):                     # keep routing fixed under the perturbations below
        margin.enforce_margin(w, inp, margin=0.08)
        regrid(w, inp)
        if margin.min_topk_gap(oracle.gate_logits(inp["x"], inp["w_gate"], inp["b_gate"]), w.k).min() >= 0.07:
            return w, inp
    raise AssertionError("could not condition the workload")


@pytest.mark.parametrize("act", [wl.ACT_GELU_ERF, wl.ACT_GELU_TANH, wl.ACT_IDENTITY])
def test_analytic_gradients_match_finite_differences(act):
    w, inp = _conditioned(act, T=10, d=9, r=5, h=7, E=4, k=2)
    _, rt = _loss(inp, w)
    grads = oracle.backward_full(inp, rt, act)
    analytic = {"x": grads["dx"], "w_gate": grads["dw_gate"], "b_gate": grads["db_gate"],
                "w_down": grads["dw_down"], "w_up": grads["dw_up"],
                "w1": np.stack([grads["dw1"][e] for e in range(w.E)]),
                "w2": np.stack([grads["dw2"][e] for e in range(w.E)])}
    g = np.random.default_rng(3)
    delta = 2.0 ** -8
    for key, an in analytic.items():
        scale = np.sqrt(np.mean(an ** 2))
        assert scale > 0
        flat = g.choice(an.size, size=min(an.size, 12), replace=False)
        for f in flat:
            index = np.unravel_index(f, an.shape)
            fd = _fd4(inp, w, key, index, delta)
            assert abs(fd - an[index]) <= 2e-7 * max(abs(an[index]), scale), (key, index, fd, an[index])


def test_relu_gradients_match_finite_differences_away_from_kinks():
    act = wl.ACT_RELU
    w, inp = _conditioned(act, T=10, d=9, r=5, h=7, E=4, k=2)
    _, rt = _loss(inp, w)
    grads = oracle.backward_full(inp, rt, act)
    analytic = {"x": grads["dx"], "w_down": grads["dw_down"], "w_up": grads["dw_up"],
                "w1": np.stack([grads["dw1"][e] for e in range(w.E)]),
                "w2": np.stack([grads["dw2"][e] for e in range(w.E)])}
    g = np.random.default_rng(5)
    checked = 0
    for key, an in analytic.items():
        scale = np.sqrt(np.mean(an ** 2))
        for f in g.choice(an.size, size=min(an.size, 16), replace=False):
            index = np.unravel_index(f, an.shape)
            fds = []
            for delta in (2.0 ** -12, 2.0 ** -13):
                lo = inp[key].copy(); hi = inp[key].copy()
                lo[index] -= np.float32(delta); hi[index] += np.float32(delta)
                fds.append((_loss(dict(inp, **{key: hi}), w)[0] - _loss(dict(inp, **{key: lo}), w)[0]) / (2 * delta))
            if abs(fds[0] - fds[1]) > 1e-6 * max(abs(fds[1]), scale):
                continue                   # a ReLU kink lies inside the stencil
            checked += 1
            assert abs(fds[1] - an[index]) <= 1e-5 * max(abs(an[index]), scale), (key, index)
    assert checked >= 40


def test_adjoint_identity_for_dx():
    w, inp = _conditioned(wl.ACT_GELU_ERF, T=8, d=9, r=5, h=7, E=4, k=2)
    _, rt = _loss(inp, w)
    dx = oracle.backward_tokens(inp, rt, w.act)["dx"]
    g = np.random.default_rng(11)
    v = (np.round(g.standard_normal(inp["x"].shape) * 4) / 4).astype(np.float32)
    delta = 2.0 ** -9
    vals = [_loss(dict(inp, x=(inp["x"] + np.float32(m * delta) * v).astype(np.float32)), w)[0] for m in (2, 1, -1, -2)]
    directional = (-vals[0] + 8 * vals[1] - 8 * vals[2] + vals[3]) / (12 * delta)
    assert abs(directional - float(np.sum(dx * v))) <= 1e-7 * abs(directional)


def test_experts_without_tokens_get_exactly_zero_gradients():
    w, inp = small_workload(T=3, E=8, k=1)
    rt = oracle.route(inp, 1)
    grads = oracle.backward_full(inp, rt, w.act)
    empty = [e for e in range(w.E) if rt.counts[e] == 0]
    assert len(empty) >= 5
    for e in empty:
        assert not grads["dw1"][e].any() and not grads["dw2"][e].any() and not grads["dw_gate"][e].any()
    assert any(grads["dw1"][e].any() for e in range(w.E))


def test_gate_gradients_sum_to_zero_per_token_and_vanish_for_k1():
    w, inp = small_workload(T=12, E=5, k=3)
    dl = oracle.backward_tokens(inp, oracle.route(inp, 3), w.act)["dlogit"]
    np.testing.assert_allclose(dl.sum(axis=1), 0.0, rtol=0, atol=1e-12)   # softmax weights sum to one
    dl1 = oracle.backward_tokens(inp, oracle.route(inp, 1), w.act)["dlogit"]
    np.testing.assert_array_equal(dl1, np.zeros_like(dl1))                # p = 1 is constant


# ---------------------------------------------------------------- closed forms of Table 3 / Eq. 1

def _golden():
    out = {}
    with open(os.path.join(GOLDEN, "table4.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                key, val = line.split()
                out[key] = float(val)
    return out


def test_table3_formulas_reproduce_table4():
    gold = _golden()
    h, l, s, e, r, top_k, ep = 2048, 24, 2048, 64, 0.25, 8, 32
    bs = 0.5 * 2 ** 20
    pf, pb = counts.params(h, l, 50257, e, r, False), counts.params(h, l, 50257, e, r, True)
    ff, fb = counts.flops(bs, s, h, l, 50304, r, top_k, False), counts.flops(bs, s, h, l, 50304, r, top_k, True)
    af, ab = counts.a2a_bytes(bs, h, l, top_k, ep, r, False), counts.a2a_bytes(bs, h, l, top_k, ep, r, True)
    assert round(pf / 1e9, 2) == gold["params_fine_grained_1e9"] and round(pb / 1e9, 2) == gold["params_bigmac_1e9"]
    assert round((pb / pf - 1) * 100, 2) == gold["params_increase_pct"]
    assert round(ff / 1e12, 2) == gold["flops_fine_grained_1e12"] and round(fb / 1e12, 2) == gold["flops_bigmac_1e12"]
    assert round((fb / ff - 1) * 100, 2) == gold["flops_increase_pct"]
    assert round(af / 2 ** 30, 2) == gold["a2a_fine_grained_GiB"] and round(ab / 2 ** 30, 2) == gold["a2a_bigmac_GiB"]
    assert round((1 - ab / af) * 100, 2) == gold["a2a_decrease_pct"]
    # Eq. 1 against Table 3's byte row: 2 passes x 2 bytes x l layers
    assert counts.layer_a2a_elements(bs, h, top_k, ep) * 2 * 2 * l == af
    assert counts.layer_a2a_elements(bs, h, top_k, ep, r) * 2 * 2 * l == ab


def test_margin_conditioning_reaches_the_requested_gap():
    w = wl.WORKLOADS["tiny"]
    inp = wl.make_inputs(w)
    margin.enforce_margin(w, inp, 1e-3)
    gaps = margin.min_topk_gap(oracle.gate_logits(inp["x"], inp["w_gate"]), w.k)
    assert gaps.min() >= 1e-3
    inp2 = wl.make_inputs(w)
    margin.enforce_margin(w, inp2, 1e-3)
    np.testing.assert_array_equal(inp["x"], inp2["x"])                    # seeded: reproducible


# ---------------------------------------------------------------- non-finite logits; the bf16 ReLU' decision

def test_topk_with_non_finite_logits_stays_in_range():
    """NaN is ordered as -inf; a round that finds only -inf takes the lowest id not yet chosen; gate values are the
    softmax of what was kept (exp(-inf) = 0), and 1/k each when nothing finite was kept.  Expected values by hand."""
    ninf, nan = -np.inf, np.nan
    logits = np.array([
        [0.5, ninf, 2.0, ninf, ninf],      # two finite experts, k = 3: 2, 0, then the lowest masked id 1
        [nan, nan, nan, nan, nan],         # a NaN token: experts 0, 1, 2 at 1/3 each
        [nan, 1.0, ninf, 1.0, 3.0],        # NaN behind every finite value; the tie 1 = 1 goes to the lower id
        [ninf, ninf, ninf, ninf, 7.0],     # one finite expert: it takes all the weight
    ])
    idx, p = oracle.topk(logits, 3)
    np.testing.assert_array_equal(idx, [[2, 0, 1], [0, 1, 2], [4, 1, 3], [4, 0, 1]])
    a = np.exp(-1.5)
    b = np.exp(-2.0)
    np.testing.assert_allclose(p[0], [1 / (1 + a), a / (1 + a), 0.0], rtol=0, atol=1e-15)
    np.testing.assert_allclose(p[1], [1 / 3, 1 / 3, 1 / 3], rtol=0, atol=1e-15)
    np.testing.assert_allclose(p[2], [1 / (1 + 2 * b), b / (1 + 2 * b), b / (1 + 2 * b)], rtol=0, atol=1e-15)
    np.testing.assert_allclose(p[3], [1.0, 0.0, 0.0], rtol=0, atol=0)
    idx5, p5 = oracle.topk(logits, 5)                      # k = E: a permutation of all experts, whatever the values
    assert all(sorted(row) == [0, 1, 2, 3, 4] for row in idx5.tolist())
    np.testing.assert_array_equal(idx5[0], [2, 0, 1, 3, 4])
    # finite rows are untouched by the rule
    g = np.random.default_rng(5)
    fin = g.standard_normal((20, 9))
    np.testing.assert_array_equal(oracle.topk(fin, 4)[0], np.argsort(-fin, axis=1, kind="stable")[:, :4].astype(np.int32))


def test_relu_decision_from_bf16_rounded_low_width_token():
    """decide_bf16: ReLU' = [z > 0] is taken from z = bf16(x') W1^T (the numbers a BF16 kernel holds), everything
    else stays exact.  E = 1, k = 1, identity descend projection, so x' = x; the first token is built so that one
    hidden unit's exact z is 2^-10 > 0 while the rounded x' gives z = 0: its decision flips.  Checked against a numpy
    restatement (library matmuls, the mask written out) and against the exact decision."""
    d = r = 4
    h, T = 5, 6
    g = np.random.default_rng(11)
    x = np.round(g.standard_normal((T, d)) * 64) / 64                      # exact in bf16 except the engineered row
    x[0] = [1.0 + 2.0 ** -10, -1.0, 0.25, -0.5]
    w1 = np.round(g.standard_normal((1, h, r)) * 8) / 8
    w1[0, 0] = [1.0, 1.0, 0.0, 0.0]                                          # z = 2^-10 exactly; 0 from bf16(x')
    w1[0, 1] = [1.0, -1.0, 0.0, 0.0]                                         # z = 2 + 2^-10: positive either way
    inp = {"x": x.astype(np.float32), "dy": g.standard_normal((T, d)).astype(np.float32),
           "w_gate": np.zeros((1, d), np.float32), "b_gate": None, "w_down": np.eye(r, d, dtype=np.float32),
           "w1": w1.astype(np.float32), "w2": g.standard_normal((1, r, h)).astype(np.float32),
           "w_up": g.standard_normal((d, r)).astype(np.float32)}
    rt = oracle.route(inp, 1)
    np.testing.assert_array_equal(rt.topk_p, 1.0)

    def restated(x_for_decision):
        X, W1, W2, Wup = _f64(inp["x"]), _f64(inp["w1"][0]), _f64(inp["w2"][0]), _f64(inp["w_up"])
        mask = (x_for_decision @ W1.T > 0).astype(np.float64)               # [T,h]
        dy_lo = _f64(inp["dy"]) @ Wup                                         # [T,r]
        dz = (dy_lo @ W2) * mask                                              # du = dy' (p = 1); da = du W2
        dx = dz @ W1                                                          # dx' = dz W1, dx = dx' I
        dw1 = dz.T @ X                                                        # x' = x
        a = np.maximum(X @ W1.T, 0.0)
        dw2 = dy_lo.T @ a
        return mask, dx, dw1, dw2

    x_rounded = _f64(wl.bf16_round(inp["x"]))
    mask_r, dx_r, dw1_r, dw2_r = restated(x_rounded)
    mask_e, dx_e, dw1_e, dw2_e = restated(_f64(inp["x"]))
    assert mask_e[0, 0] == 1.0 and mask_r[0, 0] == 0.0                       # the engineered unit flips
    assert (mask_e != mask_r).sum() == 1 and mask_e[0, 1] == mask_r[0, 1] == 1.0
    got_r = oracle.backward_full(inp, rt, wl.ACT_RELU, decide_bf16=True)
    got_e = oracle.backward_full(inp, rt, wl.ACT_RELU, decide_bf16=False)
    for got, (dx, dw1, dw2) in ((got_r, (dx_r, dw1_r, dw2_r)), (got_e, (dx_e, dw1_e, dw2_e))):
        np.testing.assert_allclose(got["dx"], dx, rtol=0, atol=1e-12)
        np.testing.assert_allclose(got["dw1"][0], dw1, rtol=0, atol=1e-12)
        np.testing.assert_allclose(got["dw2"][0], dw2, rtol=0, atol=1e-12)
    assert np.abs(got_r["dx"][0] - got_e["dx"][0]).max() > 1e-3              # the flip is visible in the gradient
    np.testing.assert_array_equal(got_r["dw2"][0], got_e["dw2"][0])          # sigma itself is never rounded
    # other activations ignore the switch
    a1 = oracle.backward_full(inp, rt, wl.ACT_GELU_ERF, decide_bf16=True)
    a0 = oracle.backward_full(inp, rt, wl.ACT_GELU_ERF, decide_bf16=False)
    np.testing.assert_array_equal(a1["dx"], a0["dx"])
