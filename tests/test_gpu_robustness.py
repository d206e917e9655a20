"""Run-to-run reproducibility: no kernel of the layer sums in an order that depends on scheduling (no floating-point
atomics; the dynamically scheduled weight-gradient kernel hands out work items at run time but every output element
is produced by one item, and the parts of a split expert are added in a fixed order), so two runs on the same inputs
must agree bit for bit, whatever ran on the GPU in between."""
import pytest

from paper_2502_16927_b200 import workloads as wl

from helpers import empty_grads, make_layer, to_device
from test_gpu_parity import conditioned

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("case", [
    dict(shape=dict(T=6000, d=256, r=256, h=512, E=16, k=2), flags=wl.FLAG_DYNAMIC_WGRAD, kw=dict()),
    dict(shape=dict(T=5000, d=256, r=128, h=256, E=24, k=3), flags=0, kw=dict(capacity_factor=1.0, aux_loss_coef=5.0)),
    dict(shape=dict(T=3000, d=128, r=64, h=128, E=8, k=2), flags=0, kw=dict(), bias=True),
])
def test_two_runs_agree_bit_for_bit(case):
    import numpy as np
    import torch

    w = wl.Workload("det", dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=131, expert_bias=case.get("bias", False), **case["shape"])
    inp = conditioned(w)
    inp["b_gate"] = (3.0 * np.linspace(1.0, -1.0, w.E) ** 3).astype(np.float32)       # long and short segments
    dev = to_device(w, inp)
    runs = []
    for attempt in range(2):
        layer = make_layer(w, case["flags"], **case["kw"])
        y = layer.forward(dev["x"], dev, training=True)
        G = empty_grads(w, "cuda", fill=float("nan"))
        dx = layer.backward(dev["x"], dev["dy"], dev, G)
        torch.cuda.synchronize()
        assert layer.status() == 0
        runs.append(dict(G, y=y.clone(), dx=dx.clone()))
        layer.close()
        if attempt == 0:                                   # disturb the GPU's state between the runs
            junk = torch.randn(4096, 4096, device="cuda")
            (junk @ junk).sum().item()
    for key, val in runs[0].items():
        assert torch.equal(val.view(torch.uint8), runs[1][key].view(torch.uint8)), key


def test_a_wait_that_runs_out_is_reported_and_leaves_the_handle_usable():
    """Failure path of the device-side waits, made without a fault: a one-thread kernel polls, with the pipelines'
    bounded wait and a short limit, a barrier nobody arrives at; it gives up, records that in the status word and
    returns.  The host reads BIGMAC_ERR_TIMEOUT once; the same handle then computes a correct step."""
    import numpy as np
    import torch

    import oracle
    from paper_2502_16927_b200 import binding
    from helpers import to_numpy

    w = wl.Workload("to", T=300, d=128, r=64, h=128, E=8, k=2, dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=139)
    inp = conditioned(w)
    dev = to_device(w, inp)
    layer = make_layer(w)
    assert layer.status() == 0
    binding.bigmac_debug_expire_wait(layer.handle)
    assert layer.status() == -5                            # BIGMAC_ERR_TIMEOUT
    assert layer.status() == 0                             # cleared by the read
    y = layer.forward(dev["x"], dev, training=False)
    torch.cuda.synchronize()
    assert layer.status() == 0
    ref = oracle.forward_tokens(inp, oracle.route(inp, w.k), w.act)["y"]
    assert oracle.max_rel_err(to_numpy(y), ref) <= 1e-2
    layer.close()


GUARD = 4096


def _guarded(nbytes, like=None, shape=None, dtype=None):
    """A buffer of exactly nbytes with GUARD bytes of 0xA5 on both sides; returns (whole, interior view)."""
    import torch

    whole = torch.full((GUARD + nbytes + GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
    inner = whole[GUARD:GUARD + nbytes]
    if dtype is not None:
        inner = inner.view(dtype).view(shape)
    return whole, inner


def _intact(whole, nbytes):
    return bool((whole[:GUARD] == 0xA5).all()) and bool((whole[GUARD + nbytes:] == 0xA5).all())


@pytest.mark.parametrize("case", [
    dict(shape=dict(T=333, d=40, r=12, h=20, E=7, k=3), dtype=wl.DTYPE_F32, kw=dict()),
    dict(shape=dict(T=1000, d=128, r=64, h=192, E=12, k=5), dtype=wl.DTYPE_BF16, kw=dict()),
    dict(shape=dict(T=2500, d=256, r=256, h=512, E=16, k=2), dtype=wl.DTYPE_BF16, kw=dict(capacity_factor=1.0, aux_loss_coef=2.0)),
    dict(shape=dict(T=700, d=128, r=128, h=256, E=8, k=2), dtype=wl.DTYPE_BF16, kw=dict(), bias=True),
])
def test_no_kernel_writes_outside_the_buffers_it_was_given(case):
    """Every buffer of a training forward + backward is given at exactly the size the library asks for, between guard
    bands; a store past either end of any of them (workspaces, saved state, outputs, gradients, tables) would change a
    guard byte without necessarily faulting."""
    import numpy as np
    import torch

    from paper_2502_16927_b200 import binding

    w = wl.Workload("gb", dtype=case["dtype"], act=wl.ACT_GELU_ERF, seed=149, expert_bias=case.get("bias", False), **case["shape"])
    inp = conditioned(w)
    inp["b_gate"] = (2.0 * np.linspace(1.0, -1.0, w.E) ** 3).astype(np.float32)
    dev = to_device(w, inp)
    layer = make_layer(w, **case["kw"])
    tdt = torch.float32 if w.dtype == wl.DTYPE_F32 else torch.bfloat16
    es = 4 if w.dtype == wl.DTYPE_F32 else 2
    s_bytes, v_bytes = binding.bigmac_workspace_bytes(layer.handle, w.T, True)
    held = {}

    def buf(name, nbytes, shape=None, dtype=None):
        whole, inner = _guarded(nbytes, shape=shape, dtype=dtype)
        held[name] = (whole, nbytes)
        return inner

    scratch, saved = buf("scratch", s_bytes), buf("saved", v_bytes)
    y = buf("y", w.T * w.d * es, (w.T, w.d), tdt)
    dx = buf("dx", w.T * w.d * es, (w.T, w.d), tdt)
    N = w.T * w.k
    R = {"topk_idx": buf("topk_idx", 4 * N, (N,), torch.int32), "topk_w": buf("topk_w", 4 * N, (N,), torch.float32),
         "counts": buf("counts", 4 * w.E, (w.E,), torch.int32), "offsets": buf("offsets", 4 * (w.E + 1), (w.E + 1,), torch.int32),
         "row_of_slot": buf("row_of_slot", 4 * N, (N,), torch.int32), "slot_of_row": buf("slot_of_row", 4 * N, (N,), torch.int32),
         "counts_chosen": buf("counts_chosen", 4 * w.E, (w.E,), torch.int32), "aux_loss": buf("aux_loss", 4, (1,), torch.float32)}
    shapes = {"dw_gate": (w.E, w.d), "dw_down": (w.r, w.d), "dw1": (w.E, w.h, w.r), "dw2": (w.E, w.r, w.h), "dw_up": (w.d, w.r)}
    G = {key: buf(key, int(np.prod(shp)) * es, shp, tdt) for key, shp in shapes.items()}
    G["db_gate"] = buf("db_gate", 4 * w.E, (w.E,), torch.float32)
    if w.expert_bias:
        G["db1"] = buf("db1", 4 * w.E * w.h, (w.E, w.h), torch.float32)
        G["db2"] = buf("db2", 4 * w.E * w.r, (w.E, w.r), torch.float32)
    binding.bigmac_forward(layer.handle, dev["x"], w.T, dev, y, R, saved, scratch)
    binding.bigmac_backward(layer.handle, dev["x"], dev["dy"], w.T, dev, saved, dx, G, False, scratch)
    torch.cuda.synchronize()
    assert layer.status() == 0
    for name, (whole, nbytes) in held.items():
        assert _intact(whole, nbytes), name
    assert bool(torch.isfinite(y.float()).all()) and bool(torch.isfinite(dx.float()).all())
    layer.close()


def test_expert_parallel_exchange_stays_inside_the_exchange_buffers():
    """The puts of every rank land inside the owners' buffers of exactly bigmac_ep_buffer_bytes, also when one rank's
    experts receive nearly all rows: guard bands around all sixteen buffers stay intact."""
    import numpy as np
    import torch

    from paper_2502_16927_b200 import ep

    w = wl.Workload("gb", T=1200, d=128, r=64, h=128, E=8, k=2, dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=151)
    inp = conditioned(w)
    b = np.full(w.E, -6.0, dtype=np.float32)
    b[:2] = 6.0                                             # everybody's two choices are rank 0's experts
    inp["b_gate"] = b
    dev = to_device(w, inp)
    size, Tq = 4, 300
    held = []

    def alloc(nbytes):
        whole, inner = _guarded(nbytes)
        held.append((whole, nbytes))
        return inner

    group = ep.EpLocalGroup(w.d, w.r, w.h, w.E, w.k, Tq, w.dtype, w.act, ["cuda"] * size, alloc=alloc)
    Ws = [ep.shard_weights(dev, q, size) for q in range(size)]
    xs = [dev["x"][q * Tq:(q + 1) * Tq].contiguous() for q in range(size)]
    dys = [dev["dy"][q * Tq:(q + 1) * Tq].contiguous() for q in range(size)]
    ys = group.forward(xs, Ws)
    Gs = [{"dw_gate": torch.empty_like(dev["w_gate"]), "dw_down": torch.empty_like(dev["w_down"]), "dw_up": torch.empty_like(dev["w_up"]),
           "dw1": torch.empty_like(Ws[q]["w1"]), "dw2": torch.empty_like(Ws[q]["w2"]),
           "db_gate": torch.empty(w.E, dtype=torch.float32, device="cuda")} for q in range(size)]
    group.backward(xs, dys, Ws, Gs)
    torch.cuda.synchronize()
    assert group.status() == 0
    assert len(held) == 4 * size
    for whole, nbytes in held:
        assert _intact(whole, nbytes)
    counts = group.ranks[0].counts_all.sum(dim=0)
    assert int(counts[:2].sum()) == w.T * w.k               # all rows went to rank 0's first two experts
    assert bool(torch.isfinite(torch.cat(ys).float()).all())
    group.close()


@pytest.mark.parametrize("variant", [{}, {"gate_low": True}, {"expert_bias": True}], ids=["plain", "gate_low", "expert_bias"])
def test_backward_on_two_streams_equals_backward_on_one_and_can_be_captured(variant):
    """bigmac_backward forks a few independent launches to the handle's second stream and joins them back: the
    results are bit for bit those of the one-stream order (the "overlap" debug switch off), a
    captured forward + backward replays to the same bits, and a pass that accumulates adds each gradient once.
    The variants put more on the second stream (the expert-bias column sums) or join it elsewhere (gate on x')."""
    import numpy as np
    import torch

    w = wl.Workload("ov", T=3000, d=256, r=128, h=256, E=16, k=4, dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=167,
                    **variant)
    inp = wl.make_inputs(w) if variant else conditioned(w)
    dev = to_device(w, inp)
    layer = make_layer(w)
    y = layer.forward(dev["x"], dev, training=True)
    G = empty_grads(w, "cuda", fill=float("nan"))
    dx = layer.backward(dev["x"], dev["dy"], dev, G)
    torch.cuda.synchronize()
    assert layer.status() == 0
    eager = {key: val.clone() for key, val in dict(G, y=y, dx=dx).items()}

    # accumulation on top of 0.5: every gradient is added exactly once (fp32 ones to rounding, BF16 ones to a BF16 step)
    G3 = empty_grads(w, "cuda", fill=0.5)
    layer.forward(dev["x"], dev, training=True)
    layer.backward(dev["x"], dev["dy"], dev, G3, accumulate=True)
    torch.cuda.synchronize()
    for key, val in G3.items():
        want = eager[key].double() + 0.5
        tol = (1e-5 if val.dtype == torch.float32 else 1e-2) * (1.0 + want.abs())
        assert bool(((val.double() - want).abs() <= tol).all()), key
        assert float(eager[key].double().abs().max()) > 0.05, key          # large enough for a second addition to show

    # the same step captured into a CUDA graph and replayed
    side = torch.cuda.Stream()
    G2 = empty_grads(w, "cuda", fill=float("nan"))
    y2, dx2 = torch.empty_like(y), torch.empty_like(dx)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        layer.forward(dev["x"], dev, y=y2, training=True)             # warm-up on the capture stream
        layer.backward(dev["x"], dev["dy"], dev, G2, dx=dx2)
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            layer.forward(dev["x"], dev, y=y2, training=True)
            layer.backward(dev["x"], dev["dy"], dev, G2, dx=dx2)
    for t in list(G2.values()) + [y2, dx2]:
        t.fill_(float("nan")) if t.is_floating_point() else None
    graph.replay()
    torch.cuda.synchronize()
    assert layer.status() == 0
    for key, val in dict(G2, y=y2, dx=dx2).items():
        assert torch.equal(val.view(torch.uint8), eager[key].view(torch.uint8)), key
    layer.close()

    # one-stream order: the same step with the overlap switch off
    from paper_2502_16927_b200 import binding

    binding.bigmac_debug_set("overlap", 0)
    try:
        layer = make_layer(w)
        y1 = layer.forward(dev["x"], dev, training=True)
        G1 = empty_grads(w, "cuda", fill=float("nan"))
        dx1 = layer.backward(dev["x"], dev["dy"], dev, G1)
        torch.cuda.synchronize()
        assert layer.status() == 0
        one = {key: val.cpu() for key, val in dict(G1, y=y1, dx=dx1).items()}
        layer.close()
    finally:
        binding.bigmac_debug_set("defaults")
    for key, val in eager.items():
        assert torch.equal(val.cpu().view(torch.uint8), one[key].view(torch.uint8)), key


@pytest.mark.parametrize("case", [
    dict(T=3000, d=256, r=128, h=256, E=16, k=4, training=True),      # a training step: every kernel of both passes
    dict(T=300, d=512, r=128, h=256, E=12, k=3, training=False),      # inference: split descend, experts on CTA pairs
])
def test_chained_launches_equal_plain_launches(case):
    """Every kernel of a call is launched with programmatic stream serialisation (it may be set up while its
    predecessor still runs and waits for it before touching memory).  Results are bit for bit those of plain
    launches (the "chain" debug switch off), also when the call is repeated back to back without a synchronisation
    in between (the next call's first kernels are then set up while this call's last ones run)."""
    import torch
    from paper_2502_16927_b200 import binding

    case = dict(case)
    training = case.pop("training")
    w = wl.Workload("chain", dtype=wl.DTYPE_BF16, act=wl.ACT_GELU_ERF, seed=421, **case)
    inp = conditioned(w)
    dev = to_device(w, inp)

    def run(repeats):
        layer = make_layer(w)
        out = None
        for _ in range(repeats):
            if training:
                y = layer.forward(dev["x"], dev, training=True)
                G = empty_grads(w, "cuda", fill=float("nan"))
                dx = layer.backward(dev["x"], dev["dy"], dev, G)
                out = dict(G, y=y, dx=dx)
            else:
                out = {"y": layer.forward(dev["x"], dev, training=False)}
        torch.cuda.synchronize()
        assert layer.status() == 0
        out = {key: val.cpu() for key, val in out.items()}
        layer.close()
        return out

    chained = run(3)
    binding.bigmac_debug_set("chain", 0)
    try:
        plain = run(1)
    finally:
        binding.bigmac_debug_set("defaults")
    for key, val in chained.items():
        assert torch.equal(val.view(torch.uint8), plain[key].view(torch.uint8)), key


@pytest.mark.parametrize("case", [
    dict(dtype=wl.DTYPE_F32, shape=dict(T=200, d=32, r=16, h=24, E=8, k=3)),               # generic top-k kernel
    dict(dtype=wl.DTYPE_BF16, shape=dict(T=700, d=128, r=64, h=128, E=64, k=8)),            # four-tokens-per-warp kernel, three-pass sort
    dict(dtype=wl.DTYPE_BF16, shape=dict(T=9, d=128, r=64, h=128, E=32, k=4), decode=True), # one-kernel small-batch forward
])
def test_non_finite_logits_keep_every_expert_id_in_range(case):
    """A NaN token and a gate bias that masks all but k - 1 experts with -inf: every id the routing writes lies in
    [0, E) (NaN ordered as -inf, lowest id not yet chosen when only -inf is left), the tables equal the oracle's bit
    for bit, masked experts get the gate value 0, the NaN token 1/k, the status word stays clean and the other tokens'
    outputs are the oracle's."""
    import numpy as np
    import torch

    import oracle
    from helpers import to_numpy
    from test_gpu_parity import check_routing

    w = wl.Workload("nf", dtype=case["dtype"], act=wl.ACT_GELU_ERF, seed=151, **case["shape"])
    inp = wl.make_inputs(w)
    finite = np.arange(w.E - w.k + 1, w.E)                                   # k - 1 experts stay finite
    b = np.full(w.E, -np.inf, dtype=np.float32)
    b[finite] = 40.0 * np.arange(1, finite.size + 1, dtype=np.float32)      # far apart: their order is the bias order
    inp["b_gate"] = b
    bad = min(3, w.T - 1)
    inp["x"][bad, :] = np.nan
    dev = to_device(w, inp)
    layer = make_layer(w)
    if case.get("decode"):
        y, R = layer.forward(dev["x"], dev, training=False, want_routing=True)
    else:
        y, R = layer.forward(dev["x"], dev, training=True, want_routing=True)
        G = empty_grads(w, "cuda", fill=float("nan"))
        layer.backward(dev["x"], dev["dy"], dev, G)
    torch.cuda.synchronize()
    assert layer.status() == 0
    idx = to_numpy(R["topk_idx"]).reshape(w.T, w.k)
    assert idx.min() >= 0 and idx.max() < w.E
    for name in ("row_of_slot", "slot_of_row"):
        t = to_numpy(R[name])
        assert t.min() >= 0 and t.max() < w.T * w.k
    rt = oracle.route(inp, w.k)
    check_routing(R, rt)
    p = to_numpy(R["topk_w"]).reshape(w.T, w.k)
    np.testing.assert_array_equal(idx[bad], np.arange(w.k))                 # the NaN token: lowest ids, equal shares
    np.testing.assert_allclose(p[bad], 1.0 / w.k, rtol=0, atol=1e-6)
    good = np.array([t for t in range(w.T) if t != bad])
    np.testing.assert_array_equal(idx[good, -1], 0)                          # last slot: the lowest masked id, weight 0
    np.testing.assert_array_equal(p[good, -1], 0.0)
    got = to_numpy(y)
    assert np.isnan(got[bad]).all() and not np.isnan(got[good]).any()
    ref = oracle.forward_tokens(inp, rt, w.act, tokens=good)["y"]
    if w.dtype == wl.DTYPE_F32:
        assert oracle.rel_err(got[good], ref) <= 1e-4
    else:
        assert oracle.max_rel_err(got[good], ref) <= 1e-2 and oracle.fro_rel_err(got[good], ref) <= 8e-3
    layer.close()
