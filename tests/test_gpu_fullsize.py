"""Parity at BASELINE's full sizes, in the launch configuration bench.py times (same handle, same calls):
the large workload (T=32768, d=4096, r=512, E=128, k=8, h=2048) and the medium one (Zipf-skewed routing).

The oracle cannot evaluate 10^12 multiply-adds, so:
  * every integer table is compared in full, bit for bit (gate logits are the only cost);
  * y and dx are compared on sampled tokens, which the oracle evaluates one by one;
  * every weight gradient is compared IN FULL through a second backward whose upstream gradient dy is zero
    outside the sampled tokens: then each weight gradient is a sum over the sampled tokens only, which the
    oracle computes from those tokens alone, while the kernels still run their full-size launches; dx must
    then be exactly zero outside the sample.
"""
import numpy as np
import pytest

import oracle
from oracle import margin
from paper_2502_16927_b200 import workloads as wl

from helpers import empty_grads, make_layer, to_device, to_numpy
from test_gpu_parity import assert_within, check_routing, float_errors

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,n_sample", [("medium", 192), ("large", 160)])
def test_full_size_sampled(name, n_sample):
    import torch

    w = wl.WORKLOADS[name]
    inp = wl.make_inputs(w)
    margin.enforce_margin(w, inp, 1e-3)
    rt = oracle.route(inp, w.k)
    rng = np.random.default_rng(w.seed)
    sample = np.sort(rng.choice(w.T, size=n_sample, replace=False)).astype(np.int32)
    # make sure the sample reaches the busiest and the least busy expert
    for e in (int(np.argmax(rt.counts)), int(np.argmin(np.where(rt.counts > 0, rt.counts, 1 << 30)))):
        rows = rt.slot_of_row[rt.offsets[e]:rt.offsets[e + 1]] // w.k
        sample = np.union1d(sample, rows[:2]).astype(np.int32)

    dev = to_device(w, inp)
    layer = make_layer(w)
    y, R = layer.forward(dev["x"], dev, training=True, want_routing=True)
    G = empty_grads(w, "cuda", fill=float("nan"))
    dx = layer.backward(dev["x"], dev["dy"], dev, G)
    torch.cuda.synchronize()
    assert layer.status() == 0
    check_routing(R, rt)                                                   # all tables, full size, bit-exact

    # sampled rows of y and dx against the per-token oracle
    ref_f = oracle.forward_tokens(inp, rt, w.act, tokens=sample)
    ref_b = oracle.backward_tokens(inp, rt, w.act, tokens=sample)
    idx = torch.from_numpy(sample.astype(np.int64)).cuda()
    got = {"y": to_numpy(y[idx]), "dx": to_numpy(dx[idx])}
    assert_within(w, float_errors(w, got, {"y": ref_f["y"], "dx": ref_b["dx"]}))
    for key in ("dw_gate", "dw_down", "dw1", "dw2", "dw_up", "db_gate"):  # full backward produced finite values
        assert bool(torch.isfinite(G[key].float()).all()), key

    # second backward: dy zero outside the sample -> every weight gradient depends on the sample only
    dy_masked = torch.zeros_like(dev["dy"])
    dy_masked[idx] = dev["dy"][idx]
    layer.forward(dev["x"], dev, training=True)
    G2 = empty_grads(w, "cuda", fill=float("nan"))
    dx2 = layer.backward(dev["x"], dy_masked, dev, G2)
    torch.cuda.synchronize()
    assert layer.status() == 0
    sub = dict(inp, x=np.ascontiguousarray(inp["x"][sample]), dy=np.ascontiguousarray(inp["dy"][sample]))
    rt_sub = oracle.route(sub, w.k)
    np.testing.assert_array_equal(rt_sub.topk_idx, rt.topk_idx[sample])
    ref = oracle.backward_full(sub, rt_sub, w.act)
    ref["dw1"] = np.stack([ref["dw1"][e] for e in range(w.E)])
    ref["dw2"] = np.stack([ref["dw2"][e] for e in range(w.E)])
    keys = ("dw_up", "dw_down", "dw_gate", "dw1", "dw2", "db_gate")
    got2 = {key: to_numpy(G2[key]) for key in keys}
    got2["dx"] = to_numpy(dx2[idx])
    assert_within(w, float_errors(w, got2, ref))
    outside = torch.ones(w.T, dtype=torch.bool, device="cuda")
    outside[idx] = False
    assert not bool(dx2[outside].any())                                    # exactly zero where dy is zero
    untouched = [e for e in range(w.E) if not np.isin(rt.topk_idx[sample], e).any()]
    for e in untouched[:8]:
        assert not got2["dw1"][e].any() and not got2["dw2"][e].any()
    layer.close()


def test_full_size_medium_with_the_pre_training_settings():
    """Medium workload (Zipf-skewed gate) under Table 5's capacity factor 1.2 and a load-balancing loss: every table in
    full (more than half of the slots are dropped), the loss value, and y / dx on sampled tokens, dx including the
    gradient of the loss (coefficient chosen so that it is as large as the layer's own gradient)."""
    import torch

    w = wl.WORKLOADS["medium"]
    f, alpha = 1.2, 40000.0
    inp = wl.make_inputs(w)
    margin.enforce_margin(w, inp, 1e-3)
    rt = oracle.route(inp, w.k, capacity_factor=f)
    assert 0.3 < 1.0 - rt.keep.mean() < 0.7
    rng = np.random.default_rng(w.seed + 1)
    sample = np.sort(rng.choice(w.T, size=160, replace=False)).astype(np.int32)
    dev = to_device(w, inp)
    layer = make_layer(w, capacity_factor=f, aux_loss_coef=alpha)
    y, R = layer.forward(dev["x"], dev, training=True, want_routing=True)
    G = empty_grads(w, "cuda", fill=float("nan"))
    dx = layer.backward(dev["x"], dev["dy"], dev, G)
    torch.cuda.synchronize()
    assert layer.status() == 0
    check_routing(R, rt)
    loss, dl_aux = oracle.aux_loss(rt.logits, rt.topk_idx, alpha)
    assert abs(R["aux_loss"].item() - loss) <= 1e-5 * loss
    ref_f = oracle.forward_tokens(inp, rt, w.act, tokens=sample)
    ref_b = oracle.backward_tokens(inp, rt, w.act, tokens=sample)
    ref_dx = ref_b["dx"] + dl_aux[sample] @ np.asarray(inp["w_gate"], dtype=np.float64)
    assert np.abs(dl_aux[sample] @ np.asarray(inp["w_gate"], dtype=np.float64)).max() > 0.05 * np.abs(ref_b["dx"]).max()
    idx = torch.from_numpy(sample.astype(np.int64)).cuda()
    got = {"y": to_numpy(y[idx]), "dx": to_numpy(dx[idx])}
    assert_within(w, float_errors(w, got, {"y": ref_f["y"], "dx": ref_dx}))
    for key in ("dw_gate", "dw_down", "dw1", "dw2", "dw_up", "db_gate"):
        assert bool(torch.isfinite(G[key].float()).all()), key
    layer.close()


def test_full_size_large_on_four_expert_parallel_ranks():
    """The large workload split over four expert-parallel ranks (8192 tokens and 32 experts each, driven on one GPU):
    the gathered counts against the oracle's of the whole batch, y and dx on sampled tokens of every rank."""
    import torch
    from paper_2502_16927_b200 import ep

    w = wl.WORKLOADS["large"]
    size, Tq = 4, w.T // 4
    inp = wl.make_inputs(w)
    margin.enforce_margin(w, inp, 1e-3)
    rt = oracle.route(inp, w.k)
    rng = np.random.default_rng(w.seed + 2)
    sample = np.sort(rng.choice(w.T, size=128, replace=False)).astype(np.int32)
    dev = to_device(w, inp)
    Ws = [ep.shard_weights(dev, q, size) for q in range(size)]
    xs = [dev["x"][q * Tq:(q + 1) * Tq] for q in range(size)]
    dys = [dev["dy"][q * Tq:(q + 1) * Tq] for q in range(size)]
    group = ep.EpLocalGroup(w.d, w.r, w.h, w.E, w.k, Tq, w.dtype, w.act, ["cuda"] * size)
    ys = group.forward(xs, Ws)
    Gs = []
    for q in range(size):
        G = {key: torch.empty_like(dev[key[1:]]) for key in ("dw_gate", "dw_down", "dw_up")}
        G.update(dw1=torch.empty_like(Ws[q]["w1"]), dw2=torch.empty_like(Ws[q]["w2"]),
                 db_gate=torch.empty(w.E, dtype=torch.float32, device="cuda"))
        Gs.append(G)
    dxs = group.backward(xs, dys, Ws, Gs)
    torch.cuda.synchronize()
    assert group.status() == 0
    np.testing.assert_array_equal(to_numpy(group.ranks[0].counts_all).sum(axis=0), rt.counts)
    np.testing.assert_array_equal(to_numpy(group.ranks[3].counts_all), to_numpy(group.ranks[0].counts_all))
    ref_f = oracle.forward_tokens(inp, rt, w.act, tokens=sample)
    ref_b = oracle.backward_tokens(inp, rt, w.act, tokens=sample)
    idx = torch.from_numpy(sample.astype(np.int64)).cuda()
    got = {"y": to_numpy(torch.cat(ys)[idx]), "dx": to_numpy(torch.cat(dxs)[idx])}
    assert_within(w, float_errors(w, got, {"y": ref_f["y"], "dx": ref_b["dx"]}))
    for G in Gs:
        for key, val in G.items():
            assert bool(torch.isfinite(val.float()).all()), key
    group.close()
