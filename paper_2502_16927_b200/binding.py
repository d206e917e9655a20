"""ctypes binding of libbigmac's C ABI (include/bigmac.h): same names, argument marshalling only.

Every step of the layer runs inside the library's CUDA kernels; torch is used here for device
memory and streams.  There is no fallback: if the shared library is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libbigmac.so")

BIGMAC_OK = 0
BIGMAC_F32, BIGMAC_BF16 = 0, 1
BIGMAC_FLAG_SIMT_GEMM = 1


class bigmac_config_t(C.Structure):
    _fields_ = ([(n, C.c_int32) for n in ("d", "r", "h", "E", "k", "max_tokens", "dtype", "act")] + [("flags", C.c_uint32)] +
                [("capacity_factor", C.c_double), ("aux_loss_coef", C.c_double)])


class bigmac_weights_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_gate", "b_gate", "w_down", "w1", "w2", "w_up", "b1", "b2")]


class bigmac_grads_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("dw_gate", "db_gate", "dw_down", "dw1", "dw2", "dw_up", "db1", "db2")]


_ROUTING_FIELDS = ("topk_idx", "topk_w", "counts", "offsets", "row_of_slot", "slot_of_row", "counts_chosen", "aux_loss")


class bigmac_routing_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _ROUTING_FIELDS]


class bigmac_debug_gemm_t(C.Structure):
    _fields_ = ([(n, C.c_void_p) for n in ("A", "B", "C", "Z")] + [(n, C.c_int64) for n in ("lda", "ldb", "ldc")] +
                [(n, C.c_int32) for n in ("M", "N", "K", "a_kmajor", "b_kmajor", "out_f32", "accumulate", "epilogue",
                                          "act", "group", "num_experts")] +
                [(n, C.c_int64) for n in ("b_stride", "c_stride")] +
                [(n, C.c_void_p) for n in ("tile_expert", "n_tiles", "poffsets")])


BIGMAC_PROFILE_SLOTS = 32


class bigmac_profile_t(C.Structure):
    _fields_ = [("launches", C.c_uint64), ("dropped", C.c_uint32), ("n_slots", C.c_int32),
                ("ms", C.c_float * BIGMAC_PROFILE_SLOTS), ("calls", C.c_uint32 * BIGMAC_PROFILE_SLOTS)]


BIGMAC_EP_MAX_RANKS = 8


class bigmac_ep_t(C.Structure):
    _fields_ = [("rank", C.c_int32), ("size", C.c_int32), ("counts_all", C.c_void_p)] + \
               [(n, C.c_void_p * BIGMAC_EP_MAX_RANKS) for n in ("xg", "u", "du", "dxg")]


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Load libbigmac.so (built in-tree by paper_2502_16927_b200/build.py); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2502_16927_b200.build` first")
        L = C.CDLL(LIB_PATH)
        vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
        L.bigmac_layer_create.argtypes = [C.POINTER(bigmac_config_t), C.POINTER(vp)]
        L.bigmac_layer_destroy.argtypes = [vp]
        L.bigmac_workspace_bytes.argtypes = [vp, i32, C.c_int, C.POINTER(sz), C.POINTER(sz)]
        L.bigmac_route.argtypes = [vp, vp, i32, C.POINTER(bigmac_weights_t), C.POINTER(bigmac_routing_t), vp, sz, vp]
        L.bigmac_forward.argtypes = [vp, vp, i32, C.POINTER(bigmac_weights_t), vp, C.POINTER(bigmac_routing_t), vp,
                                     vp, sz, vp]
        L.bigmac_backward.argtypes = [vp, vp, vp, i32, C.POINTER(bigmac_weights_t), vp, vp, C.POINTER(bigmac_grads_t),
                                      C.c_int, vp, sz, vp]
        L.bigmac_device_status.argtypes = [vp, vp]
        L.bigmac_status_string.argtypes = [C.c_int]
        L.bigmac_status_string.restype = C.c_char_p
        L.bigmac_exchange_rows.argtypes = [vp, vp, i32, i32, vp, vp, sz, vp, C.c_int, vp]
        L.bigmac_debug_gemm.argtypes = [vp, C.POINTER(bigmac_debug_gemm_t), C.c_int, vp]
        L.bigmac_debug_expire_wait.argtypes = [vp, vp]
        L.bigmac_debug_expire_wait.restype = C.c_int
        L.bigmac_debug_set.argtypes = [C.c_char_p, C.c_int]
        L.bigmac_debug_set.restype = C.c_int
        L.bigmac_route_static.argtypes = [vp, vp, i32, C.POINTER(bigmac_weights_t), C.POINTER(bigmac_routing_t), vp]
        L.bigmac_route_static.restype = C.c_int
        L.bigmac_profile_enable.argtypes = [vp, C.c_int]
        L.bigmac_profile_read.argtypes = [vp, vp, C.POINTER(bigmac_profile_t)]
        L.bigmac_profile_slot_name.argtypes = [C.c_int]
        L.bigmac_profile_slot_name.restype = C.c_char_p
        W, R, G, EP = (C.POINTER(t) for t in (bigmac_weights_t, bigmac_routing_t, bigmac_grads_t, bigmac_ep_t))
        L.bigmac_ep_buffer_bytes.argtypes = [vp, i32, C.POINTER(sz)]
        L.bigmac_ep_workspace_bytes.argtypes = [vp, i32, i32, C.POINTER(sz), C.POINTER(sz)]
        L.bigmac_ep_route.argtypes = [vp, vp, i32, W, EP, R, vp, vp, sz, vp]
        L.bigmac_ep_dispatch.argtypes = [vp, i32, EP, vp, vp]
        L.bigmac_ep_experts.argtypes = [vp, W, EP, vp, vp]
        L.bigmac_ep_combine.argtypes = [vp, i32, W, EP, vp, vp, vp]
        L.bigmac_ep_backward_combine.argtypes = [vp, vp, i32, W, EP, G, C.c_int, vp, vp, sz, vp]
        L.bigmac_ep_backward_experts.argtypes = [vp, W, EP, G, C.c_int, vp, vp, sz, vp]
        L.bigmac_ep_backward_dispatch.argtypes = [vp, vp, i32, W, EP, vp, G, C.c_int, vp, vp, sz, vp]
        for name in ("bigmac_ep_buffer_bytes", "bigmac_ep_workspace_bytes", "bigmac_ep_route", "bigmac_ep_dispatch",
                     "bigmac_ep_experts", "bigmac_ep_combine", "bigmac_ep_backward_combine", "bigmac_ep_backward_experts",
                     "bigmac_ep_backward_dispatch"):
            getattr(L, name).restype = C.c_int
        for name in ("bigmac_profile_enable", "bigmac_profile_read", "bigmac_layer_create", "bigmac_layer_destroy", "bigmac_workspace_bytes", "bigmac_route",
                     "bigmac_forward", "bigmac_backward", "bigmac_device_status", "bigmac_exchange_rows",
                     "bigmac_debug_gemm"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


class BigmacError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().bigmac_status_string(status).decode()} ({status})")


def _check(status: int, where: str) -> None:
    if status != BIGMAC_OK:
        raise BigmacError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors passed to libbigmac must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


# ---- the C ABI, name for name -------------------------------------------------------------------------

def bigmac_layer_create(d, r, h, E, k, max_tokens, dtype, act, flags=0, capacity_factor=0.0, aux_loss_coef=0.0) -> C.c_void_p:
    cfg = bigmac_config_t(d, r, h, E, k, max_tokens, dtype, act, flags, capacity_factor, aux_loss_coef)
    handle = C.c_void_p()
    _check(lib().bigmac_layer_create(C.byref(cfg), C.byref(handle)), "bigmac_layer_create")
    return handle


def bigmac_layer_destroy(handle) -> None:
    _check(lib().bigmac_layer_destroy(handle), "bigmac_layer_destroy")


def bigmac_workspace_bytes(handle, T: int, training: bool):
    s, v = C.c_size_t(), C.c_size_t()
    _check(lib().bigmac_workspace_bytes(handle, T, int(training), C.byref(s), C.byref(v)), "bigmac_workspace_bytes")
    return s.value, v.value


def _weights(W: Dict[str, torch.Tensor]) -> bigmac_weights_t:
    # w_down / w_up are absent for the projection-free layer (BIGMAC_FLAG_CDAC)
    return bigmac_weights_t(_ptr(W.get("w_gate")), _ptr(W.get("b_gate")), _ptr(W.get("w_down")), _ptr(W.get("w1")),
                            _ptr(W.get("w2")), _ptr(W.get("w_up")), _ptr(W.get("b1")), _ptr(W.get("b2")))


def _grads(G: Dict[str, torch.Tensor]) -> bigmac_grads_t:
    return bigmac_grads_t(*[_ptr(G.get(n)) for n in ("dw_gate", "db_gate", "dw_down", "dw1", "dw2", "dw_up", "db1", "db2")])


def _routing(R: Optional[Dict[str, torch.Tensor]]):
    if R is None:
        return None
    return C.byref(bigmac_routing_t(*[_ptr(R.get(n)) for n in _ROUTING_FIELDS]))


def bigmac_route(handle, x, T, W, routing, scratch) -> None:
    _check(lib().bigmac_route(handle, _ptr(x), T, C.byref(_weights(W)), _routing(routing), _ptr(scratch),
                              scratch.numel() * scratch.element_size(), _stream()), "bigmac_route")


def bigmac_route_static(handle, x, T, W, routing) -> None:
    """bigmac_route without a scratch buffer: intermediates live in the library's fixed device array
    (BIGMAC_STATIC_SCRATCH_BYTES).  For callers that cannot allocate device memory; raises BigmacError with
    status -7 if (T, E, k) does not fit.  Calls must not overlap on the GPU (they share the array)."""
    _check(lib().bigmac_route_static(handle, _ptr(x), T, C.byref(_weights(W)), _routing(routing), _stream()),
           "bigmac_route_static")


def bigmac_forward(handle, x, T, W, y, routing, saved, scratch) -> None:
    _check(lib().bigmac_forward(handle, _ptr(x), T, C.byref(_weights(W)), _ptr(y), _routing(routing), _ptr(saved),
                                _ptr(scratch), scratch.numel() * scratch.element_size(), _stream()), "bigmac_forward")


def bigmac_backward(handle, x, dy, T, W, saved, dx, G, accumulate, scratch) -> None:
    _check(lib().bigmac_backward(handle, _ptr(x), _ptr(dy), T, C.byref(_weights(W)), _ptr(saved), _ptr(dx),
                                 C.byref(_grads(G)), int(accumulate), _ptr(scratch),
                                 scratch.numel() * scratch.element_size(), _stream()), "bigmac_backward")


def bigmac_device_status(handle) -> int:
    return lib().bigmac_device_status(handle, _stream())


def bigmac_exchange_rows(handle, saved, T, width, src, grouped, dst, which) -> None:
    _check(lib().bigmac_exchange_rows(handle, _ptr(saved), T, width, _ptr(src), _ptr(grouped),
                                      grouped.numel() * grouped.element_size(), _ptr(dst), which, _stream()),
           "bigmac_exchange_rows")


def bigmac_profile_enable(handle, on: bool) -> None:
    _check(lib().bigmac_profile_enable(handle, int(on)), "bigmac_profile_enable")


def bigmac_profile_read(handle) -> Dict[str, object]:
    """Synchronises the current stream; returns {"launches", "dropped", "stages": {name: (ms, calls)}}."""
    prof = bigmac_profile_t()
    _check(lib().bigmac_profile_read(handle, _stream(), C.byref(prof)), "bigmac_profile_read")
    stages = {lib().bigmac_profile_slot_name(i).decode(): (float(prof.ms[i]), int(prof.calls[i]))
              for i in range(prof.n_slots) if prof.calls[i]}
    return {"launches": int(prof.launches), "dropped": int(prof.dropped), "stages": stages}


def bigmac_debug_gemm(handle, q: bigmac_debug_gemm_t, use_tensor_cores) -> None:
    """use_tensor_cores: False/0 plain FMA, True/1 tensor cores, 2 one-CTA kernel, 3/4/5 CTA-pair kernel with 4/2/1 working
    epilogue warps per lane quadrant."""
    _check(lib().bigmac_debug_gemm(handle, C.byref(q), int(use_tensor_cores), _stream()), "bigmac_debug_gemm")


def bigmac_debug_set(name: str, value: int = 0) -> None:
    """Process-wide measurement / debugging switch ("overlap", "tc_pair", "groupk", "fused_mlp", "epi_parts",
    "staged_stores", "fuse_dispatch", "tc_mask"; "defaults" restores all).  The defaults are the product."""
    _check(lib().bigmac_debug_set(name.encode(), int(value)), "bigmac_debug_set")


def bigmac_debug_expire_wait(handle) -> None:
    """Launch the one-thread kernel whose bounded wait runs out (failure path of the device-side waits)."""
    _check(lib().bigmac_debug_expire_wait(handle, _stream()), "bigmac_debug_expire_wait")


# ---- expert parallelism: the phase calls, name for name ----------------------------------------------------

def bigmac_ep_buffer_bytes(handle, size: int) -> int:
    n = C.c_size_t()
    _check(lib().bigmac_ep_buffer_bytes(handle, size, C.byref(n)), "bigmac_ep_buffer_bytes")
    return n.value


def bigmac_ep_workspace_bytes(handle, T: int, size: int):
    s, v = C.c_size_t(), C.c_size_t()
    _check(lib().bigmac_ep_workspace_bytes(handle, T, size, C.byref(s), C.byref(v)), "bigmac_ep_workspace_bytes")
    return s.value, v.value


def make_ep(rank: int, size: int, counts_all: torch.Tensor, ptrs: Dict[str, list]) -> bigmac_ep_t:
    """ptrs[name][q]: device address (int) of rank q's exchange buffer `name` as this rank addresses it."""
    ep = bigmac_ep_t()
    ep.rank, ep.size, ep.counts_all = rank, size, counts_all.data_ptr()
    for name in ("xg", "u", "du", "dxg"):
        arr = getattr(ep, name)
        for q in range(size):
            arr[q] = ptrs[name][q]
    return ep


def _nbytes(t: torch.Tensor) -> int:
    return t.numel() * t.element_size()


def bigmac_ep_route(handle, x, T, W, ep, routing, saved, scratch) -> None:
    _check(lib().bigmac_ep_route(handle, _ptr(x), T, C.byref(_weights(W)), C.byref(ep), _routing(routing), _ptr(saved),
                                 _ptr(scratch), _nbytes(scratch), _stream()), "bigmac_ep_route")


def bigmac_ep_dispatch(handle, T, ep, saved) -> None:
    _check(lib().bigmac_ep_dispatch(handle, T, C.byref(ep), _ptr(saved), _stream()), "bigmac_ep_dispatch")


def bigmac_ep_experts(handle, W, ep, saved) -> None:
    _check(lib().bigmac_ep_experts(handle, C.byref(_weights(W)), C.byref(ep), _ptr(saved), _stream()), "bigmac_ep_experts")


def bigmac_ep_combine(handle, T, W, ep, y, saved) -> None:
    _check(lib().bigmac_ep_combine(handle, T, C.byref(_weights(W)), C.byref(ep), _ptr(y), _ptr(saved), _stream()),
           "bigmac_ep_combine")


def bigmac_ep_backward_combine(handle, dy, T, W, ep, G, accumulate, saved, scratch) -> None:
    _check(lib().bigmac_ep_backward_combine(handle, _ptr(dy), T, C.byref(_weights(W)), C.byref(ep), C.byref(_grads(G)),
                                            int(accumulate), _ptr(saved), _ptr(scratch), _nbytes(scratch), _stream()),
           "bigmac_ep_backward_combine")


def bigmac_ep_backward_experts(handle, W, ep, G, accumulate, saved, scratch) -> None:
    _check(lib().bigmac_ep_backward_experts(handle, C.byref(_weights(W)), C.byref(ep), C.byref(_grads(G)), int(accumulate),
                                            _ptr(saved), _ptr(scratch), _nbytes(scratch), _stream()),
           "bigmac_ep_backward_experts")


def bigmac_ep_backward_dispatch(handle, x, T, W, ep, dx, G, accumulate, saved, scratch) -> None:
    _check(lib().bigmac_ep_backward_dispatch(handle, _ptr(x), T, C.byref(_weights(W)), C.byref(ep), _ptr(dx),
                                             C.byref(_grads(G)), int(accumulate), _ptr(saved), _ptr(scratch),
                                             _nbytes(scratch), _stream()), "bigmac_ep_backward_dispatch")


# ---- a small convenience wrapper: owns the handle and the workspaces ------------------------------------

class Layer:
    """One BigMac layer handle plus torch-allocated workspaces.  Marshalling only."""

    def __init__(self, d, r, h, E, k, max_tokens, dtype, act, flags=0, device="cuda", capacity_factor=0.0, aux_loss_coef=0.0):
        self.cfg = dict(d=d, r=r, h=h, E=E, k=k, max_tokens=max_tokens, dtype=dtype, act=act, flags=flags,
                        capacity_factor=capacity_factor, aux_loss_coef=aux_loss_coef)
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self.handle = bigmac_layer_create(d, r, h, E, k, max_tokens, dtype, act, flags, capacity_factor, aux_loss_coef)
        self.tdtype = torch.bfloat16 if dtype == BIGMAC_BF16 else torch.float32
        self._scratch = None
        self._saved = None
        self._T = None

    def close(self):
        if self.handle is not None:
            bigmac_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _workspaces(self, T, training):
        s, v = bigmac_workspace_bytes(self.handle, T, training)
        if self._scratch is None or self._scratch.numel() < s:
            self._scratch = torch.empty(max(s, 256), dtype=torch.uint8, device=self.device)
        if training and (self._saved is None or self._saved.numel() < v):
            self._saved = torch.empty(max(v, 256), dtype=torch.uint8, device=self.device)

    def empty_routing(self, T):
        E, k = self.cfg["E"], self.cfg["k"]
        i32 = dict(dtype=torch.int32, device=self.device)
        return {"topk_idx": torch.empty(T * k, **i32), "topk_w": torch.empty(T * k, dtype=torch.float32, device=self.device),
                "counts": torch.empty(E, **i32), "offsets": torch.empty(E + 1, **i32),
                "row_of_slot": torch.empty(T * k, **i32), "slot_of_row": torch.empty(T * k, **i32),
                "counts_chosen": torch.empty(E, **i32), "aux_loss": torch.empty(1, dtype=torch.float32, device=self.device)}

    def route(self, x, W):
        T = x.shape[0]
        self._workspaces(T, False)
        R = self.empty_routing(T)
        bigmac_route(self.handle, x, T, W, R, self._scratch)
        return R

    def forward(self, x, W, y=None, training=False, want_routing=False):
        T = x.shape[0]
        self._workspaces(T, training)
        if y is None:
            y = torch.empty_like(x)
        R = self.empty_routing(T) if want_routing else None
        bigmac_forward(self.handle, x, T, W, y, R, self._saved if training else None, self._scratch)
        self._T = T if training else None
        return (y, R) if want_routing else y

    def backward(self, x, dy, W, G, dx=None, accumulate=False):
        T = x.shape[0]
        if self._T != T:
            raise RuntimeError("backward needs a training forward of the same batch first")
        if dx is None:
            dx = torch.empty_like(x)
        bigmac_backward(self.handle, x, dy, T, W, self._saved, dx, G, accumulate, self._scratch)
        return dx

    def status(self) -> int:
        return bigmac_device_status(self.handle)
