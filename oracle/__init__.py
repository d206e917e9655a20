"""numpy front end of the CPU oracle for the BigMac DCCA MoE layer.  TEST INFRASTRUCTURE ONLY.

Thin ctypes marshalling over oracle/bigmac_oracle.cpp (fp64, per token / per row, written from
Eq. 2 and Eq. 4 of the paper).  Nothing under the product package may import this module; only the
tests, the smoke check and the benchmark's CPU-baseline leg do.

Float inputs are float32 arrays holding values exactly representable in the workload dtype; every
result is float64 or int32.  Weights are [out_features, in_features].
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np

from . import build as _build

_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


@dataclass
class Routing:
    logits: np.ndarray        # [T,E] f64
    topk_idx: np.ndarray      # [T,k] int32, slots in descending-logit order
    topk_p: np.ndarray        # [T,k] f64, softmax over the k selected logits
    counts: np.ndarray        # [E]   int32
    offsets: np.ndarray       # [E+1] int32, exclusive prefix sum of counts
    row_of_slot: np.ndarray   # [T*k] int32 (-1: dropped under a capacity limit)
    slot_of_row: np.ndarray   # [T*k] int32 (-1 past the kept rows)
    keep: Optional[np.ndarray] = None            # [T*k] uint8, None = dropless
    counts_chosen: Optional[np.ndarray] = None   # [E] int32: slots that chose e, before dropping
    gate_low: bool = False                       # the gate read x' (w_gate is [E,r]) instead of x


def gate_logits(x, w_gate, b_gate=None) -> np.ndarray:
    x, w_gate = _f32(x), _f32(w_gate)
    b = None if b_gate is None else _f32(b_gate)
    T, d = x.shape
    E = w_gate.shape[0]
    out = np.empty((T, E), dtype=np.float64)
    lib().oracle_gate_logits(_p(x), _p(w_gate), _p(b), C.c_int(T), C.c_int(d), C.c_int(E), _p(out))
    return out


def gate_logits_low(x, w_down, w_gate, b_gate=None, round_x_lo_bf16: bool = False) -> np.ndarray:
    """Gate logits when the gate reads x' = x W'_down (w_gate [E,r]); x' optionally rounded to bf16 first."""
    x, w_down, w_gate = _f32(x), _f32(w_down), _f32(w_gate)
    b = None if b_gate is None else _f32(b_gate)
    T, d = x.shape
    E, r = w_gate.shape
    out = np.empty((T, E), dtype=np.float64)
    lib().oracle_gate_logits_low(_p(x), _p(w_down), _p(w_gate), _p(b), C.c_int(T), C.c_int(d), C.c_int(r), C.c_int(E),
                                 C.c_int(int(round_x_lo_bf16)), _p(out))
    return out


def topk(logits: np.ndarray, k: int):
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    T, E = logits.shape
    assert 1 <= k <= E
    idx = np.empty((T, k), dtype=np.int32)
    p = np.empty((T, k), dtype=np.float64)
    lib().oracle_topk(_p(logits), C.c_int(T), C.c_int(E), C.c_int(k), _p(idx), _p(p))
    return idx, p


def tables(topk_idx: np.ndarray, E: int):
    topk_idx = np.ascontiguousarray(topk_idx, dtype=np.int32)
    T, k = topk_idx.shape
    counts = np.empty(E, dtype=np.int32)
    offsets = np.empty(E + 1, dtype=np.int32)
    row_of_slot = np.empty(T * k, dtype=np.int32)
    slot_of_row = np.empty(T * k, dtype=np.int32)
    lib().oracle_tables(_p(topk_idx), C.c_int(T), C.c_int(k), C.c_int(E), _p(counts), _p(offsets),
                        _p(row_of_slot), _p(slot_of_row))
    return counts, offsets, row_of_slot, slot_of_row


def capacity_rows(T: int, k: int, E: int, capacity_factor: float) -> int:
    """C = ceil(f T k / E) rows per expert (Table 5's capacity factor f), evaluated in double as (f * (T k)) / E."""
    return int(np.ceil(float(capacity_factor) * float(T * k) / float(E)))


def tables_capacity(topk_idx: np.ndarray, E: int, cap: int):
    topk_idx = np.ascontiguousarray(topk_idx, dtype=np.int32)
    T, k = topk_idx.shape
    chosen = np.empty(E, dtype=np.int32)
    counts = np.empty(E, dtype=np.int32)
    offsets = np.empty(E + 1, dtype=np.int32)
    row_of_slot = np.empty(T * k, dtype=np.int32)
    slot_of_row = np.empty(T * k, dtype=np.int32)
    keep = np.empty(T * k, dtype=np.uint8)
    lib().oracle_tables_capacity(_p(topk_idx), C.c_int(T), C.c_int(k), C.c_int(E), C.c_int(cap), _p(chosen),
                                 _p(counts), _p(offsets), _p(row_of_slot), _p(slot_of_row), _p(keep))
    return chosen, counts, offsets, row_of_slot, slot_of_row, keep


def aux_loss(logits: np.ndarray, topk_idx: np.ndarray, alpha: float, want_grad: bool = True):
    """Load-balancing loss L_aux (Table 5, coefficient alpha) and dL_aux/dlogits [T,E]."""
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    topk_idx = np.ascontiguousarray(topk_idx, dtype=np.int32)
    T, E = logits.shape
    loss = C.c_double(0.0)
    grad = np.empty((T, E), dtype=np.float64) if want_grad else None
    lib().oracle_aux_loss(_p(logits), _p(topk_idx), C.c_int(T), C.c_int(E), C.c_int(topk_idx.shape[1]),
                          C.c_double(alpha), C.byref(loss), _p(grad))
    return loss.value, grad


def route(inp: Dict[str, np.ndarray], k: int, capacity_factor: float = 0.0, gate_low: bool = False,
          round_x_lo_bf16: bool = False) -> Routing:
    if gate_low:
        logits = gate_logits_low(inp["x"], inp["w_down"], inp["w_gate"], inp.get("b_gate"), round_x_lo_bf16)
    else:
        logits = gate_logits(inp["x"], inp["w_gate"], inp.get("b_gate"))
    idx, p = topk(logits, k)
    T, E = logits.shape
    if capacity_factor > 0:
        chosen, counts, offsets, ros, sor, keep = tables_capacity(idx, E, capacity_rows(T, k, E, capacity_factor))
        return Routing(logits, idx, p, counts, offsets, ros, sor, keep, chosen, gate_low)
    counts, offsets, ros, sor = tables(idx, E)
    return Routing(logits, idx, p, counts, offsets, ros, sor, None, counts.copy(), gate_low)


def _bias(inp, key):
    """Expert bias b1 [E,h] / b2 [E,r] as float32, or None (Eq. 4 has none; they are a variant)."""
    b = inp.get(key)
    return None if b is None else _f32(b)


def _dims(inp):
    T, d = inp["x"].shape
    E, h, r = inp["w1"].shape
    return T, d, r, h, E


def _tokens(tokens, T):
    if tokens is None:
        return None, T
    tok = np.ascontiguousarray(tokens, dtype=np.int32)
    assert tok.ndim == 1 and (tok.size == 0 or (tok.min() >= 0 and tok.max() < T))
    return tok, tok.size


def forward_tokens(inp, routing: Routing, act: int, tokens=None, want_slots: bool = False):
    """Per-token evaluation of Eq. 2.  Returns x_lo [n,r], y_lo [n,r], y [n,d] (+ z [n,k,h], u [n,k,r])."""
    T, d, r, h, E = _dims(inp)
    k = routing.topk_idx.shape[1]
    tok, n = _tokens(tokens, T)
    x_lo = np.empty((n, r)); y_lo = np.empty((n, r)); y = np.empty((n, d))
    z = np.empty((n, k, h)) if want_slots else None
    u = np.empty((n, k, r)) if want_slots else None
    lib().oracle_forward_tokens(_p(_f32(inp["x"])), _p(_f32(inp["w_down"])), _p(_f32(inp["w1"])),
                                _p(_f32(inp["w2"])), _p(_f32(inp["w_up"])), _p(routing.topk_idx),
                                _p(routing.topk_p), _p(tok), C.c_int(n), C.c_int(d), C.c_int(r), C.c_int(h),
                                C.c_int(E), C.c_int(k), C.c_int(act), _p(x_lo), _p(y_lo), _p(y), _p(z), _p(u),
                                _p(routing.keep), _p(_bias(inp, "b1")), _p(_bias(inp, "b2")))
    out = {"x_lo": x_lo, "y_lo": y_lo, "y": y}
    if want_slots:
        out["z"], out["u"] = z, u
    return out


def forward_grouped(inp, routing: Routing, act: int):
    """Dispatch / per-expert segments / combine evaluation; must equal forward_tokens."""
    T, d, r, h, E = _dims(inp)
    k = routing.topk_idx.shape[1]
    xg = np.empty((T * k, r)); y_lo = np.empty((T, r)); y = np.empty((T, d))
    lib().oracle_forward_grouped(_p(_f32(inp["x"])), _p(_f32(inp["w_down"])), _p(_f32(inp["w1"])),
                                 _p(_f32(inp["w2"])), _p(_f32(inp["w_up"])), _p(routing.topk_p),
                                 _p(routing.offsets), _p(routing.row_of_slot), _p(routing.slot_of_row),
                                 C.c_int(T), C.c_int(d), C.c_int(r), C.c_int(h), C.c_int(E), C.c_int(k),
                                 C.c_int(act), _p(xg), _p(y_lo), _p(y), _p(_bias(inp, "b1")), _p(_bias(inp, "b2")))
    return {"xg": xg, "y_lo": y_lo, "y": y}


def backward_tokens(inp, routing: Routing, act: int, tokens=None, decide_bf16: bool = False):
    """Per-token gradients of L = sum(y*dy): dx [n,d], dx_lo [n,r], dlogit [n,k] (top-k slots), dy_lo [n,r].

    decide_bf16: take the ReLU' decision (z > 0) from x' rounded to bf16, as the BF16 kernels do; a
    discrete decision has to be taken on the same numbers on both sides.  No effect on other activations."""
    T, d, r, h, E = _dims(inp)
    k = routing.topk_idx.shape[1]
    tok, n = _tokens(tokens, T)
    dx = np.empty((n, d)); dx_lo = np.empty((n, r)); dlogit = np.empty((n, k)); dy_lo = np.empty((n, r))
    lib().oracle_backward_tokens(_p(_f32(inp["x"])), _p(_f32(inp["dy"])), _p(_f32(inp["w_gate"])),
                                 _p(_f32(inp["w_down"])), _p(_f32(inp["w1"])), _p(_f32(inp["w2"])),
                                 _p(_f32(inp["w_up"])), _p(routing.topk_idx), _p(routing.topk_p), _p(tok),
                                 C.c_int(n), C.c_int(d), C.c_int(r), C.c_int(h), C.c_int(E), C.c_int(k),
                                 C.c_int(act), C.c_int(int(decide_bf16)), _p(dx), _p(dx_lo), _p(dlogit), _p(dy_lo),
                                 _p(routing.keep), C.c_int(int(routing.gate_low)), _p(_bias(inp, "b1")),
                                 _p(_bias(inp, "b2")))
    return {"dx": dx, "dx_lo": dx_lo, "dlogit": dlogit, "dy_lo": dy_lo}


def backward_expert(inp, routing: Routing, act: int, e: int, decide_bf16: bool = False, want_bias_grads: bool = False):
    """dW1[e] [h,r] and dW2[e] [r,h], summed over the rows of expert e's segment (+ db1[e] [h], db2[e] [r])."""
    T, d, r, h, E = _dims(inp)
    k = routing.topk_idx.shape[1]
    dw1 = np.empty((h, r)); dw2 = np.empty((r, h))
    db1 = np.empty(h) if want_bias_grads else None
    db2 = np.empty(r) if want_bias_grads else None
    lib().oracle_backward_expert(_p(_f32(inp["x"])), _p(_f32(inp["dy"])), _p(_f32(inp["w_down"])),
                                 _p(_f32(inp["w1"])), _p(_f32(inp["w2"])), _p(_f32(inp["w_up"])),
                                 _p(routing.topk_p), _p(routing.offsets), _p(routing.slot_of_row), C.c_int(e),
                                 C.c_int(d), C.c_int(r), C.c_int(h), C.c_int(k), C.c_int(act), C.c_int(int(decide_bf16)),
                                 _p(dw1), _p(dw2), _p(_bias(inp, "b1")), _p(_bias(inp, "b2")), _p(db1), _p(db2))
    return (dw1, dw2, db1, db2) if want_bias_grads else (dw1, dw2)


def backward_full(inp, routing: Routing, act: int, experts=None, decide_bf16: bool = False, aux_alpha: float = 0.0):
    """All gradients: dx and every weight gradient (dw1/dw2 for `experts`, default all).

    aux_alpha > 0: gradients of sum(y*dy) + L_aux; the dense gate gradient dL_aux/dl [T,E] reaches dx, dw_gate and
    db_gate through the linear gate (three matrix products with it)."""
    T, d, r, h, E = _dims(inp)
    k = routing.topk_idx.shape[1]
    fwd = forward_tokens(inp, routing, act)
    bwd = backward_tokens(inp, routing, act, decide_bf16=decide_bf16)
    dw_up = np.empty((d, r)); dw_down = np.empty((r, d)); dw_gate = np.empty((E, d)); db_gate = np.empty(E)
    lib().oracle_backward_shared(_p(_f32(inp["x"])), _p(_f32(inp["dy"])), _p(fwd["y_lo"]), _p(bwd["dx_lo"]),
                                 _p(routing.topk_idx), _p(bwd["dlogit"]), C.c_int(T), C.c_int(d), C.c_int(r),
                                 C.c_int(E), C.c_int(k), _p(dw_up), _p(dw_down), _p(dw_gate), _p(db_gate))
    dw1, dw2 = {}, {}
    with_bias = inp.get("b1") is not None
    db1 = np.zeros((E, h)) if with_bias else None
    db2 = np.zeros((E, r)) if with_bias else None
    if experts is None:
        all1 = np.empty((E, h, r)); all2 = np.empty((E, r, h))
        lib().oracle_backward_all_experts(_p(_f32(inp["x"])), _p(_f32(inp["dy"])), _p(_f32(inp["w_down"])),
                                          _p(_f32(inp["w1"])), _p(_f32(inp["w2"])), _p(_f32(inp["w_up"])),
                                          _p(routing.topk_p), _p(routing.offsets), _p(routing.slot_of_row),
                                          C.c_int(E), C.c_int(d), C.c_int(r), C.c_int(h), C.c_int(k), C.c_int(act),
                                          C.c_int(int(decide_bf16)), _p(all1), _p(all2), _p(_bias(inp, "b1")),
                                          _p(_bias(inp, "b2")), _p(db1), _p(db2))
        for e in range(E):
            dw1[e], dw2[e] = all1[e], all2[e]
    else:
        for e in experts:
            if with_bias:
                dw1[e], dw2[e], db1[e], db2[e] = backward_expert(inp, routing, act, e, decide_bf16, True)
            else:
                dw1[e], dw2[e] = backward_expert(inp, routing, act, e, decide_bf16)
    out = {"y": fwd["y"], "y_lo": fwd["y_lo"], "x_lo": fwd["x_lo"], "dx": bwd["dx"], "dx_lo": bwd["dx_lo"],
           "dlogit": bwd["dlogit"], "dw_up": dw_up, "dw_down": dw_down, "dw_gate": dw_gate,
           "db_gate": db_gate, "dw1": dw1, "dw2": dw2}
    if with_bias:
        out["db1"], out["db2"] = db1, db2
    if routing.gate_low:
        # the gate read x': dW_g [E,r] = dl^T x' with dl scattered to its dense [T,E] form (a library matmul); dx' above
        # already holds the gate's share, so dw_down is complete
        assert aux_alpha == 0
        dl_dense = np.zeros((T, E))
        np.put_along_axis(dl_dense, routing.topk_idx.astype(np.int64), bwd["dlogit"], axis=1)
        out["dw_gate"] = dl_dense.T @ fwd["x_lo"]
    if aux_alpha > 0:
        loss, dl_aux = aux_loss(routing.logits, routing.topk_idx, aux_alpha)
        x64 = np.asarray(inp["x"], dtype=np.float64)
        out["aux_loss"] = loss
        out["dlogit_aux"] = dl_aux
        out["dx"] = out["dx"] + dl_aux @ np.asarray(inp["w_gate"], dtype=np.float64)    # l = x W_g^T + b_g
        out["dw_gate"] = dw_gate + dl_aux.T @ x64
        out["db_gate"] = db_gate + dl_aux.sum(axis=0)
    return out


def max_rel_err(a, b) -> float:
    """max_i |a_i - b_i| / max_i |b_i|: the largest error relative to the largest reference magnitude."""
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    if b.size == 0:
        return 0.0
    top = float(np.max(np.abs(b)))
    if top == 0.0:
        return float(np.max(np.abs(a)))
    return float(np.max(np.abs(a - b))) / top


def fro_rel_err(a, b) -> float:
    """||a - b||_F / ||b||_F."""
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    nb = float(np.linalg.norm(b))
    return float(np.linalg.norm(a - b)) / nb if nb > 0 else float(np.linalg.norm(a))


def rel_err(a, b) -> float:
    """max_i |a_i - b_i| / max(|b_i|, rms(b)): elementwise relative error with the denominator
    floored at the reference tensor's RMS, so near-zero elements do not dominate."""
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    if b.size == 0:
        return 0.0
    rms = float(np.sqrt(np.mean(b * b)))
    if rms == 0.0:
        return float(np.max(np.abs(a))) if a.size else 0.0
    return float(np.max(np.abs(a - b) / np.maximum(np.abs(b), rms)))
