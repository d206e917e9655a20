"""GPU parity of the expert-parallel layer (Fig. 2c): `size` ranks with their own tokens and E/size experts each,
exchanging r-wide rows through each other's buffers, against the CPU oracle applied to the concatenation of the
ranks' batches.  The ranks are driven by one process on one GPU (their kernels never wait on one another: every
phase of every rank is a launch of its own), which exercises the same kernels, tables and addresses as one rank
per GPU; what differs there is only that the buffer addresses are peer mappings and the barriers collectives."""
import numpy as np
import pytest

import oracle
from oracle import margin
from paper_2502_16927_b200 import binding, ep, workloads as wl

from helpers import oracle_inputs, to_device, to_numpy
from test_gpu_parity import TOL, assert_within, float_errors

pytestmark = pytest.mark.gpu


def run_group(w, inp, tokens_per_rank, flags=0):
    """Split the workload's tokens over the ranks, run forward + backward, return per-rank results and the group's sums."""
    import torch

    size = len(tokens_per_rank)
    assert sum(tokens_per_rank) == w.T
    dev = to_device(w, inp)
    full = {key: dev[key] for key in ("w_gate", "w_down", "w1", "w2", "w_up") if key in dev}
    if "b_gate" in dev:
        full["b_gate"] = dev["b_gate"]
    Ws = [ep.shard_weights(full, q, size) for q in range(size)]
    bounds = np.concatenate([[0], np.cumsum(tokens_per_rank)])
    xs = [dev["x"][bounds[q]:bounds[q + 1]].contiguous() for q in range(size)]
    dys = [dev["dy"][bounds[q]:bounds[q + 1]].contiguous() for q in range(size)]
    if w.cdac:
        flags |= wl.FLAG_CDAC
    group = ep.EpLocalGroup(w.d, w.r, w.h, w.E, w.k, max(max(tokens_per_rank), 1), w.dtype, w.act, ["cuda"] * size, flags)
    ys = group.forward(xs, Ws)
    dt = torch.float32 if w.dtype == wl.DTYPE_F32 else torch.bfloat16
    per = w.E // size
    Gs = []
    for q in range(size):
        shapes = {"dw_gate": (w.E, w.d), "dw_down": (w.r, w.d), "dw_up": (w.d, w.r), "dw1": (per, w.h, w.r), "dw2": (per, w.r, w.h)}
        if w.cdac:
            del shapes["dw_down"], shapes["dw_up"]
        G = {key: torch.full(shp, float("nan"), dtype=dt, device="cuda") for key, shp in shapes.items()}
        G["db_gate"] = torch.full((w.E,), float("nan"), dtype=torch.float32, device="cuda")
        Gs.append(G)
    dxs = group.backward(xs, dys, Ws, Gs)
    torch.cuda.synchronize()
    assert group.status() == 0
    busy = [q for q in range(size) if tokens_per_rank[q] > 0]            # a rank without tokens writes no shared gradients
    got = {"y": np.concatenate([to_numpy(y) for y in ys]), "dx": np.concatenate([to_numpy(v) for v in dxs]),
           "dw1": np.concatenate([to_numpy(G["dw1"]) for G in Gs]), "dw2": np.concatenate([to_numpy(G["dw2"]) for G in Gs]),
           "counts_all": to_numpy(group.ranks[0].counts_all)}
    for key in ep.SHARED_GRADS:
        if key in Gs[0]:
            got[key] = sum(to_numpy(Gs[q][key]) for q in busy)
    group.close()
    return got


def compare(w, inp, got):
    inp = oracle_inputs(w, inp)                     # Eq. 3 is Eq. 2 with identity projections for the oracle
    rt = oracle.route(inp, w.k)
    np.testing.assert_array_equal(got["counts_all"].sum(axis=0), rt.counts)
    ref = oracle.backward_full(inp, rt, w.act, decide_bf16=w.dtype == wl.DTYPE_BF16)
    ref["dw1"] = np.stack([ref["dw1"][e] for e in range(w.E)])
    ref["dw2"] = np.stack([ref["dw2"][e] for e in range(w.E)])
    keys = ("y", "dx", "dw_gate", "dw1", "dw2", "db_gate") + (() if w.cdac else ("dw_up", "dw_down"))
    assert_within(w, float_errors(w, {key: got[key] for key in keys}, ref))
    for e in range(w.E):
        if rt.counts[e] == 0:
            assert not got["dw1"][e].any() and not got["dw2"][e].any()


def skewed(w, strength):
    inp = wl.make_inputs(w)
    if strength:
        inp["b_gate"] = (strength * np.linspace(1.0, -1.0, w.E) ** 3).astype(np.float32)
    margin.enforce_margin(w, inp, 1e-3)
    return inp


@pytest.mark.parametrize("tokens", [[700], [400, 300], [1, 0, 650, 49], [175] * 4, [100, 50, 90, 60, 120, 80, 110, 90]])
def test_fp32_ranks_together_equal_one_layer(tokens):
    w = wl.Workload("ep", T=sum(tokens), d=64, r=24, h=40, E=8, k=3, dtype=wl.DTYPE_F32, act=wl.ACT_GELU_ERF, seed=71)
    inp = skewed(w, 1.5)
    compare(w, inp, run_group(w, inp, tokens))


@pytest.mark.parametrize("case", [
    dict(shape=dict(d=256, r=128, h=256, E=16, k=4), tokens=[1500, 1500], strength=0.0),
    dict(shape=dict(d=256, r=256, h=512, E=16, k=2), tokens=[2500, 100, 1400, 2000], strength=3.0),   # one rank's experts take most rows
    dict(shape=dict(d=128, r=64, h=128, E=24, k=3), tokens=[900, 1100, 1000], strength=2.0),         # some experts without rows
])
@pytest.mark.parametrize("flags", [0, wl.FLAG_DYNAMIC_WGRAD])
def test_bf16_ranks_together_equal_one_layer(case, flags):
    w = wl.Workload("ep", T=sum(case["tokens"]), dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=73, **case["shape"])
    inp = skewed(w, case["strength"])
    compare(w, inp, run_group(w, inp, case["tokens"], flags))


@pytest.mark.parametrize("case", [
    dict(shape=dict(d=48, r=48, h=20, E=8, k=3), dtype=wl.DTYPE_F32, tokens=[150, 0, 200, 77]),
    dict(shape=dict(d=128, r=128, h=64, E=8, k=2), dtype=wl.DTYPE_BF16, tokens=[900, 1100]),
    dict(shape=dict(d=256, r=256, h=128, E=12, k=4), dtype=wl.DTYPE_BF16, tokens=[700, 500, 800]),
])
def test_conventional_layer_of_eq3_on_expert_parallel_ranks(case):
    """BIGMAC_FLAG_CDAC under expert parallelism: the rows that travel are the tokens themselves at width d."""
    w = wl.Workload("ep", T=sum(case["tokens"]), dtype=case["dtype"], act=wl.ACT_GELU_ERF, seed=163, cdac=True, **case["shape"])
    inp = skewed(w, 1.5)
    compare(w, inp, run_group(w, inp, case["tokens"]))


@pytest.mark.parametrize("case", [
    dict(shape=dict(d=16, r=8, h=8, E=1024, k=3), dtype=wl.DTYPE_F32, tokens=[90, 70, 0, 110, 60, 80, 100, 90]),
    dict(shape=dict(d=64, r=64, h=64, E=1024, k=2), dtype=wl.DTYPE_BF16, tokens=[800, 700, 900, 600]),
])
def test_the_largest_expert_count_on_expert_parallel_ranks(case):
    """E = 1024, the most the library takes: 128 or 256 experts per rank, most of them with a handful of rows or none."""
    w = wl.Workload("ep", T=sum(case["tokens"]), dtype=case["dtype"], act=wl.ACT_GELU_ERF, seed=167, **case["shape"])
    inp = skewed(w, 0.3)
    compare(w, inp, run_group(w, inp, case["tokens"]))


def test_small_config_on_four_ranks():
    w = wl.WORKLOADS["small"]
    inp = skewed(w, 0.0)
    compare(w, inp, run_group(w, inp, [1024] * 4))


def test_unsupported_combinations_and_bad_arguments():
    w = wl.WORKLOADS["tiny"]
    for kw in (dict(capacity_factor=1.2), dict(aux_loss_coef=0.1)):
        h = binding.bigmac_layer_create(w.d, w.r, w.h, w.E, w.k, 64, w.dtype, w.act, 0, **kw)
        with pytest.raises(binding.BigmacError) as err:
            binding.bigmac_ep_buffer_bytes(h, 2)
        assert err.value.status == -2
        binding.bigmac_layer_destroy(h)
    h = binding.bigmac_layer_create(w.d, w.r, w.h, w.E, w.k, 64, w.dtype, w.act)
    for size in (0, 3, 9):                                   # E = 8: not a divisor, out of range
        with pytest.raises(binding.BigmacError) as err:
            binding.bigmac_ep_buffer_bytes(h, size)
        assert err.value.status == -1
    assert binding.bigmac_ep_buffer_bytes(h, 2) > 0
    binding.bigmac_layer_destroy(h)


def test_one_rank_per_process_plumbing_with_a_group_of_one():
    """The torch.distributed path (symmetric-memory exchange buffers, all_gather of the counts, collective barriers)
    with a process group of one rank: the same calls a multi-GPU job makes, here addressing only local memory."""
    import os
    import torch
    import torch.distributed as dist

    w = wl.Workload("ep", T=600, d=128, r=64, h=128, E=8, k=2, dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=79)
    inp = skewed(w, 1.0)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(31500 + os.getpid() % 1000))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        dev = to_device(w, inp)
        try:
            rank = ep.EpProcessRank(w.d, w.r, w.h, w.E, w.k, w.T, w.dtype, w.act)
        except (RuntimeError, NotImplementedError) as err:       # torch's symmetric memory is not available on this host
            if isinstance(err, binding.BigmacError):
                raise
            pytest.skip(f"torch symmetric memory unavailable: {err}")
        y = rank.forward(dev["x"], dev)
        G = {"dw_gate": torch.empty_like(dev["w_gate"]), "dw_down": torch.empty_like(dev["w_down"]),
             "dw_up": torch.empty_like(dev["w_up"]), "dw1": torch.empty_like(dev["w1"]), "dw2": torch.empty_like(dev["w2"]),
             "db_gate": torch.empty(w.E, dtype=torch.float32, device="cuda")}
        dx = rank.backward(dev["x"], dev["dy"], dev, G)
        torch.cuda.synchronize()
        assert rank.status() == 0
        got = {"y": to_numpy(y), "dx": to_numpy(dx), "counts_all": to_numpy(rank.rk.counts_all)}
        got.update({key: to_numpy(val) for key, val in G.items()})
        rank.close()
    finally:
        dist.destroy_process_group()
    compare(w, inp, got)


@pytest.mark.parametrize("bad", [1 << 30, -5])
def test_a_count_matrix_that_cannot_be_right_is_refused_on_the_device(bad):
    """A rank whose count matrix was not gathered properly (here: another rank's row holds impossible values) must not
    store outside the buffers: its step moves and computes nothing, the status word says so, the handle stays usable."""
    import torch

    w = wl.Workload("ep", T=400, d=64, r=24, h=40, E=8, k=3, dtype=wl.DTYPE_F32, act=wl.ACT_GELU_ERF, seed=137)
    inp = skewed(w, 1.0)
    dev = to_device(w, inp)
    Ws = [ep.shard_weights(dev, q, 2) for q in range(2)]
    xs = [dev["x"][:200].contiguous(), dev["x"][200:].contiguous()]
    dys = [dev["dy"][:200].contiguous(), dev["dy"][200:].contiguous()]
    group = ep.EpLocalGroup(w.d, w.r, w.h, w.E, w.k, 200, w.dtype, w.act, ["cuda"] * 2)
    for buf in group.ranks[0].buffers.values():
        buf.fill_(0)
    for rk in group.ranks:
        rk.route(xs[rk.rank], Ws[rk.rank])
    group.ranks[0].counts_all[1].fill_(bad)               # rank 0 never received rank 1's counts
    group.ranks[1].counts_all[0].copy_(group.ranks[0].counts_all[0])
    ys = [torch.full_like(x, float("nan")) for x in xs]
    rk0 = group.ranks[0]
    rk0.dispatch()
    rk0.experts(Ws[0])
    rk0.combine(Ws[0], ys[0])
    G = {"dw_gate": torch.empty_like(dev["w_gate"]), "dw_down": torch.empty_like(dev["w_down"]), "dw_up": torch.empty_like(dev["w_up"]),
         "dw1": torch.empty_like(Ws[0]["w1"]), "dw2": torch.empty_like(Ws[0]["w2"]),
         "db_gate": torch.empty(w.E, dtype=torch.float32, device="cuda")}
    dx = torch.empty_like(xs[0])
    rk0.backward_combine(dys[0], Ws[0], G)
    rk0.backward_experts(Ws[0], G)
    rk0.backward_dispatch(xs[0], Ws[0], dx, G)
    torch.cuda.synchronize()
    assert rk0.status() == -6                               # BIGMAC_ERR_STATE, and the word is cleared by the read
    assert rk0.status() == 0
    assert not bool(ys[0].any())                            # nothing was combined: y' = 0
    assert not bool(G["dw1"].any()) and not bool(G["dw2"].any())
    assert not bool(rk0.buffers["xg"].any()) and not bool(rk0.buffers["du"].any())     # its puts went nowhere
    # the same handles run a proper step afterwards
    got_y = group.forward(xs, Ws)
    torch.cuda.synchronize()
    assert group.status() == 0
    rt = oracle.route(inp, w.k)
    ref = oracle.forward_tokens(inp, rt, w.act)["y"]
    assert_within(w, float_errors(w, {"y": np.concatenate([to_numpy(v) for v in got_y])}, {"y": ref}))
    group.close()
