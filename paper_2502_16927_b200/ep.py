"""Expert-parallel BigMac layer (Fig. 2c): plumbing around the bigmac_ep_* phase calls.

Every rank holds the shared matrices and E/size experts; the two exchanges at the low width r are made by the
library's kernels over peer memory.  This module only allocates buffers, hands the ranks each other's buffer
addresses, gathers the per-expert counts and places the barriers between the phases:

  EpLocalGroup     all ranks live in this process (several GPUs with peer access, or several ranks on one GPU,
                   which is how the path is exercised where only one GPU is at hand): buffer addresses are used
                   directly, a barrier is an event wait between the ranks' streams.
  EpProcessRank    one rank per process under torch.distributed: exchange buffers come from symmetric memory, the
                   counts travel by all_gather, a barrier is a collective on the ranks' streams.

No arithmetic of the layer lives here.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import torch

from . import binding

SHARED_GRADS = ("dw_gate", "db_gate", "dw_down", "dw_up")       # summed over ranks by the caller (data parallel)
EXCHANGE_BUFFERS = ("xg", "u", "du", "dxg")


# ---- host-side helpers (no GPU needed) --------------------------------------------------------------------

def experts_of_rank(E: int, rank: int, size: int) -> range:
    """Rank q owns the contiguous block of E/size experts [q E/size, (q+1) E/size)."""
    if size < 1 or E % size or not 0 <= rank < size:
        raise ValueError("E must be a multiple of the number of ranks and 0 <= rank < size")
    per = E // size
    return range(rank * per, (rank + 1) * per)


def owner_of_expert(E: int, e: int, size: int) -> int:
    return e // (E // size)


def shard_weights(W: Dict[str, torch.Tensor], rank: int, size: int) -> Dict[str, torch.Tensor]:
    """This rank's view of a full weight set: shared matrices as they are, w1 / w2 cut to the owned experts."""
    own = experts_of_rank(W["w1"].shape[0], rank, size)
    out = dict(W)
    out["w1"] = W["w1"][own.start:own.stop].contiguous()
    out["w2"] = W["w2"][own.start:own.stop].contiguous()
    return out


def gather_counts(counts_all: torch.Tensor, rank: int, group=None) -> None:
    """Fill every row of counts_all [size, E] from the ranks' own rows (row `rank` holds this rank's counts)."""
    import torch.distributed as dist

    dist.all_gather_into_tensor(counts_all.view(-1), counts_all[rank].clone(), group=group)


def reduce_shared_grads(G: Dict[str, torch.Tensor], group=None) -> None:
    """Sum the shared matrices' gradients over the ranks (each rank returns the share of its own tokens)."""
    import torch.distributed as dist

    for name in SHARED_GRADS:
        if G.get(name) is not None:
            dist.all_reduce(G[name], group=group)


def placement(counts_all, rank: int, pad: int = 128):
    """The row placement the library computes on the device (a restatement for sizing and tests): counts_all
    [size, E] -> (send_base [E], poffsets of every owner [size][E/size + 1]).  Expert e lives at rank e // (E/size);
    its segment starts at the padded prefix of that rank's experts and holds rank 0's rows first, then rank 1's, ...;
    send_base[e] is where THIS rank's first row of expert e lands."""
    size, E = len(counts_all), len(counts_all[0])
    per = E // size
    total = [sum(int(counts_all[p][e]) for p in range(size)) for e in range(E)]
    poffsets = []
    for q in range(size):
        off = [0]
        for j in range(per):
            off.append(off[-1] + (total[q * per + j] + pad - 1) // pad * pad)
        poffsets.append(off)
    send_base = [poffsets[e // per][e % per] + sum(int(counts_all[p][e]) for p in range(rank)) for e in range(E)]
    return send_base, poffsets


def exchange_bytes_per_rank(T: int, k: int, width: int, size: int, elem_bytes: int) -> int:
    """Bytes one rank sends in one exchange when its slots spread evenly over the ranks (Eq. 1 per direction and
    rank: k T width (size-1)/size elements)."""
    return T * k * width * elem_bytes * (size - 1) // size


# ---- one rank ------------------------------------------------------------------------------------------------

class EpRank:
    """Handle, workspaces and exchange buffers of one rank.  `alloc(nbytes) -> uint8 tensor` provides the exchange
    buffers (symmetric memory between processes, plain device memory within one)."""

    def __init__(self, d, r, h, E, k, max_tokens, dtype, act, rank, size, device, flags=0, alloc=None):
        self.rank, self.size, self.E, self.k = rank, size, E, k
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self.handle = binding.bigmac_layer_create(d, r, h, E, k, max_tokens, dtype, act, flags)
            nbytes = binding.bigmac_ep_buffer_bytes(self.handle, size)
            alloc = alloc or (lambda n: torch.empty(n, dtype=torch.uint8, device=self.device))
            self.buffers = {name: alloc(max(nbytes, 256)) for name in EXCHANGE_BUFFERS}
            self.counts_all = torch.zeros((size, E), dtype=torch.int32, device=self.device)
        self.tdtype = torch.bfloat16 if dtype == binding.BIGMAC_BF16 else torch.float32
        self._scratch = self._saved = None
        self.ep = None
        self.T = 0

    def connect(self, ptrs: Dict[str, List[int]]) -> None:
        """ptrs[name][q]: address of rank q's buffer `name` in this rank's address space."""
        self.ep = binding.make_ep(self.rank, self.size, self.counts_all, ptrs)

    def _workspaces(self, T):
        s, v = binding.bigmac_ep_workspace_bytes(self.handle, T, self.size)
        if self._scratch is None or self._scratch.numel() < s:
            self._scratch = torch.empty(max(s, 256), dtype=torch.uint8, device=self.device)
        if self._saved is None or self._saved.numel() < v:
            self._saved = torch.empty(max(v, 256), dtype=torch.uint8, device=self.device)

    # forward phases
    def route(self, x, W, routing=None):
        self.T = x.shape[0]
        self._workspaces(self.T)
        binding.bigmac_ep_route(self.handle, x, self.T, W, self.ep, routing, self._saved, self._scratch)

    def dispatch(self):
        binding.bigmac_ep_dispatch(self.handle, self.T, self.ep, self._saved)

    def experts(self, W):
        binding.bigmac_ep_experts(self.handle, W, self.ep, self._saved)

    def combine(self, W, y):
        binding.bigmac_ep_combine(self.handle, self.T, W, self.ep, y, self._saved)

    # backward phases
    def backward_combine(self, dy, W, G, accumulate=False):
        binding.bigmac_ep_backward_combine(self.handle, dy, self.T, W, self.ep, G, accumulate, self._saved, self._scratch)

    def backward_experts(self, W, G, accumulate=False):
        binding.bigmac_ep_backward_experts(self.handle, W, self.ep, G, accumulate, self._saved, self._scratch)

    def backward_dispatch(self, x, W, dx, G, accumulate=False):
        binding.bigmac_ep_backward_dispatch(self.handle, x, self.T, W, self.ep, dx, G, accumulate, self._saved, self._scratch)

    def status(self) -> int:
        return binding.bigmac_device_status(self.handle)

    def close(self):
        if self.handle is not None:
            binding.bigmac_layer_destroy(self.handle)
            self.handle = None


# ---- all ranks in one process ----------------------------------------------------------------------------------

class EpLocalGroup:
    """`size` ranks driven by this process.  devices[q] is rank q's GPU; the same GPU may appear several times."""

    def __init__(self, d, r, h, E, k, max_tokens, dtype, act, devices: Sequence, flags=0, alloc=None):
        self.size = len(devices)
        self.ranks = [EpRank(d, r, h, E, k, max_tokens, dtype, act, q, self.size, devices[q], flags, alloc=alloc)
                      for q in range(self.size)]
        distinct = sorted({rk.device.index or 0 for rk in self.ranks})
        for a in distinct:
            for b in distinct:
                if a != b and not torch.cuda.can_device_access_peer(a, b):
                    raise RuntimeError(f"GPU {a} cannot address GPU {b}'s memory")
        ptrs = {name: [rk.buffers[name].data_ptr() for rk in self.ranks] for name in EXCHANGE_BUFFERS}
        for rk in self.ranks:
            rk.connect(ptrs)

    def _each(self, fn):
        for rk in self.ranks:
            with torch.cuda.device(rk.device):
                fn(rk)

    def barrier(self):
        """Work enqueued after this call on any rank's stream starts after all work enqueued before it on every
        rank's stream has finished."""
        events = []
        for rk in self.ranks:
            with torch.cuda.device(rk.device):
                ev = torch.cuda.Event()
                ev.record()
                events.append(ev)
        for rk in self.ranks:
            with torch.cuda.device(rk.device):
                for ev in events:
                    torch.cuda.current_stream().wait_event(ev)

    def forward(self, xs, Ws, ys=None, routings=None):
        ys = ys or [torch.empty_like(x) for x in xs]
        self._each(lambda rk: rk.route(xs[rk.rank], Ws[rk.rank], routings[rk.rank] if routings else None))
        self.barrier()
        for rk in self.ranks:                       # the all-gather of the counts: every rank's row to every rank
            with torch.cuda.device(rk.device):
                for src in self.ranks:
                    if src is not rk:
                        rk.counts_all[src.rank].copy_(src.counts_all[src.rank], non_blocking=True)
        self.barrier()
        self._each(lambda rk: rk.dispatch())
        self.barrier()
        self._each(lambda rk: rk.experts(Ws[rk.rank]))
        self.barrier()
        self._each(lambda rk: rk.combine(Ws[rk.rank], ys[rk.rank]))
        return ys

    def backward(self, xs, dys, Ws, Gs, dxs=None, accumulate=False):
        dxs = dxs or [torch.empty_like(x) for x in xs]
        self.barrier()
        self._each(lambda rk: rk.backward_combine(dys[rk.rank], Ws[rk.rank], Gs[rk.rank], accumulate))
        self.barrier()
        self._each(lambda rk: rk.backward_experts(Ws[rk.rank], Gs[rk.rank], accumulate))
        self.barrier()
        self._each(lambda rk: rk.backward_dispatch(xs[rk.rank], Ws[rk.rank], dxs[rk.rank], Gs[rk.rank], accumulate))
        return dxs

    def status(self) -> int:
        return min(rk.status() for rk in self.ranks)

    def close(self):
        for rk in self.ranks:
            rk.close()


# ---- one rank per process ------------------------------------------------------------------------------------------

class EpStepOrder:
    """Order of the phase calls of one step and of the barriers between them, for one rank per process (Fig. 2c):

        route | all-gather of counts | dispatch | experts | combine
        backward_combine | backward_experts | backward_dispatch | (sum of the shared gradients)

    "|" is a barrier over all ranks' streams: what follows reads rows that peers wrote in what precedes (experts read
    the rows every rank put; combine gets the outputs of every owner; ...).  The all-gather doubles as the barrier
    that orders a step after the previous one.  A subclass provides `rk` (the phase calls of this rank), `barrier()`,
    `gather()` (fill every row of the count matrix) and `reduce(G)` (sum the shared matrices' gradients)."""

    rk = None

    def barrier(self):
        raise NotImplementedError

    def gather(self):
        raise NotImplementedError

    def reduce(self, G):
        raise NotImplementedError

    def forward(self, x, W, y=None, routing=None):
        y = torch.empty_like(x) if y is None else y
        self.rk.route(x, W, routing)
        self.gather()                                # also orders this step after the last one
        self.rk.dispatch()
        self.barrier()
        self.rk.experts(W)
        self.barrier()
        self.rk.combine(W, y)
        return y

    def backward(self, x, dy, W, G, dx=None, accumulate=False, reduce_shared=True):
        dx = torch.empty_like(x) if dx is None else dx
        self.barrier()
        self.rk.backward_combine(dy, W, G, accumulate)
        self.barrier()
        self.rk.backward_experts(W, G, accumulate)
        self.barrier()
        self.rk.backward_dispatch(x, W, dx, G, accumulate)
        if reduce_shared:
            self.reduce(G)
        return dx


class EpProcessRank(EpStepOrder):
    """This process's rank of a torch.distributed group (NCCL): exchange buffers in symmetric memory, so that every
    rank can address every other rank's; counts by all_gather; barriers as one-element all_reduces on the ranks'
    streams.  Plain peer loads and stores only."""

    def __init__(self, d, r, h, E, k, max_tokens, dtype, act, group=None, flags=0):
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm

        self.group = group if group is not None else dist.group.WORLD
        rank, size = dist.get_rank(self.group), dist.get_world_size(self.group)
        device = torch.device("cuda", torch.cuda.current_device())
        self._handles = {}

        def alloc(nbytes):
            t = symm.empty(nbytes, dtype=torch.uint8, device=device)
            self._handles[t.data_ptr()] = symm.rendezvous(t, self.group)
            return t

        self.rk = EpRank(d, r, h, E, k, max_tokens, dtype, act, rank, size, device, flags, alloc=alloc)
        ptrs = {name: [int(p) for p in self._handles[self.rk.buffers[name].data_ptr()].buffer_ptrs]
                for name in EXCHANGE_BUFFERS}
        self.rk.connect(ptrs)
        self._flag = torch.zeros(1, dtype=torch.int32, device=device)

    def barrier(self):
        import torch.distributed as dist

        dist.all_reduce(self._flag, group=self.group)

    def gather(self):
        gather_counts(self.rk.counts_all, self.rk.rank, self.group)

    def reduce(self, G):
        reduce_shared_grads(G, self.group)

    def status(self) -> int:
        return self.rk.status()

    def close(self):
        self.rk.close()
