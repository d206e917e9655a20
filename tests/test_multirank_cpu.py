"""The N > 1 paths on CPU: two gloo ranks.  Expert parallelism: the host-side plumbing of the exchange (count
all-gather, weight sharding, gradient reduction) and the row-placement rule, checked against the oracle's tables
of the concatenated batch.  bench.py: its ranks run independent batches, so what is multi-rank there is only the
bookkeeping: per-rank seeds, the max-over-ranks of the device time, the whole-job throughput, and the reference arm
running on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 5.0 + 2.0 * rank                       # rank 1 is the slow one
    ms = bench.slowest_rank_ms(ms_local)
    out[rank] = (ms, bench.whole_job_tokens_per_s(1000, world, ms), bench.rank_seed(1237, rank))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_rank_time():
    world, port = 2, 29500 + os.getpid() % 1000
    manager = mp.Manager()
    out = manager.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0][0] == out[1][0] == 7.0
    assert out[0][1] == out[1][1] == 2 * 1000 / 7e-3
    assert out[0][2] != out[1][2]


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.slowest_rank_ms(3.5) == 3.5
    assert bench.whole_job_tokens_per_s(32768, 1, 10.0) == 32768 / 10e-3


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                        "--steps", "1", "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                        "--steps", "1", "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


# ---------------------------------------------------------------- expert parallelism: host side

def _ep_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    import oracle
    from paper_2502_16927_b200 import ep

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    E, k, T = 6, 2, (37, 20)[rank]
    g = np.random.default_rng(100 + rank)
    logits = g.standard_normal((T, E)) + np.linspace(1.5, -1.5, E)
    idx, _ = oracle.topk(logits, k)
    counts, offsets, ros, _ = oracle.tables(idx, E)
    counts_all = torch.zeros((world, E), dtype=torch.int32)
    counts_all[rank] = torch.from_numpy(counts)
    ep.gather_counts(counts_all, rank)
    send_base, poffsets = ep.placement(counts_all.tolist(), rank)
    dest = [(ep.owner_of_expert(E, int(e), world), send_base[e] + int(ros[s]) - int(offsets[e]))
            for s, e in enumerate(idx.ravel())]
    W = {"w_gate": torch.zeros(E, 4), "w1": torch.arange(E * 3 * 2, dtype=torch.float32).reshape(E, 3, 2),
         "w2": torch.arange(E * 2 * 3, dtype=torch.float32).reshape(E, 2, 3)}
    mine = ep.shard_weights(W, rank, world)
    G = {"dw_gate": torch.full((E, 4), float(rank + 1)), "db_gate": torch.full((E,), float(rank + 1)), "dw_down": None,
         "dw_up": torch.ones(4, 2), "dw1": torch.full((3,), 7.0)}
    ep.reduce_shared_grads(G)
    out[rank] = dict(idx=idx, dest=dest, counts_all=counts_all.numpy().copy(), poffsets=poffsets,
                     w1_first=float(mine["w1"][0, 0, 0]), w1_shape=tuple(mine["w1"].shape),
                     dw_gate=float(G["dw_gate"][0, 0]), db_gate=float(G["db_gate"][0]), dw1=float(G["dw1"][0]))
    dist.barrier()
    dist.destroy_process_group()


def test_expert_parallel_host_side_with_two_ranks():
    import numpy as np
    import oracle

    world, port = 2, 30500 + os.getpid() % 1000
    manager = mp.Manager()
    out = manager.dict()
    mp.spawn(_ep_worker, args=(world, port, out), nprocs=world, join=True)
    E, k, per = 6, 2, 3
    np.testing.assert_array_equal(out[0]["counts_all"], out[1]["counts_all"])           # the all-gather
    assert out[0]["poffsets"] == out[1]["poffsets"]
    # the placement: one layer over the concatenated batch (rank 0's tokens first) sorts every expert's rows the same way
    idx = np.concatenate([out[0]["idx"], out[1]["idx"]])
    counts, offsets, ros, _ = oracle.tables(idx, E)
    np.testing.assert_array_equal(out[0]["counts_all"].sum(axis=0), counts)
    dest = out[0]["dest"] + out[1]["dest"]
    seen = set()
    for s, e in enumerate(idx.ravel()):
        q, row = dest[s]
        assert q == e // per
        assert row == out[0]["poffsets"][q][e % per] + (ros[s] - offsets[e])
        assert (q, row) not in seen
        seen.add((q, row))
    # sharding and gradient reduction
    assert out[0]["w1_shape"] == out[1]["w1_shape"] == (per, 3, 2)
    assert out[0]["w1_first"] == 0.0 and out[1]["w1_first"] == float(per * 3 * 2)
    for r_ in (0, 1):
        assert out[r_]["dw_gate"] == 3.0 and out[r_]["db_gate"] == 3.0 and out[r_]["dw1"] == 7.0   # experts' gradients stay


# ---------------------------------------------------------------- expert parallelism: order of phases and barriers

# what a phase reads from its peers: every rank must have finished these before any rank starts the phase
_NEEDS_FROM_ALL = {"dispatch": ("route",), "experts": ("dispatch",), "combine": ("experts",),
                   "backward_combine": ("combine",), "backward_experts": ("backward_combine",),
                   "backward_dispatch": ("backward_experts",)}


def _order_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2502_16927_b200 import ep

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    store = dist.distributed_c10d._get_default_store()
    log, violations = [], []

    class StubRank:
        """Phase calls that do no arithmetic: each records that this rank ran it (in the store every rank sees) after
        checking that every rank has finished what the phase reads from its peers."""
        counts_all = torch.zeros((world, 4), dtype=torch.int32)

        def __init__(self):
            self.rank, self.step = rank, 0

        def _run(self, name):
            import time
            for need in _NEEDS_FROM_ALL.get(name, ()):
                for q in range(world):
                    if store.add(f"{self.step}/{need}/{q}", 0) != 1:
                        violations.append((self.step, name, need, q))
            time.sleep(0.02 * (rank + 1) if name in ("dispatch", "experts", "backward_experts") else 0.0)   # ranks drift apart
            store.add(f"{self.step}/{name}/{rank}", 1)
            log.append(name)

        def route(self, x, W, routing=None): self._run("route"); self.counts_all[rank] = rank + 1
        def dispatch(self): self._run("dispatch")
        def experts(self, W): self._run("experts")
        def combine(self, W, y): self._run("combine")
        def backward_combine(self, dy, W, G, accumulate=False): self._run("backward_combine")
        def backward_experts(self, W, G, accumulate=False): self._run("backward_experts")
        def backward_dispatch(self, x, W, dx, G, accumulate=False): self._run("backward_dispatch"); self.step += 1

    class Order(ep.EpStepOrder):
        def __init__(self):
            self.rk = StubRank()
            self._flag = torch.zeros(1, dtype=torch.int32)

        def barrier(self):
            log.append("|")
            dist.all_reduce(self._flag)

        def gather(self):
            log.append("gather")
            ep.gather_counts(self.rk.counts_all, rank)

        def reduce(self, G):
            log.append("reduce")
            ep.reduce_shared_grads(G)

    order = Order()
    x = torch.zeros(3, 4)
    G = {"dw_gate": torch.full((2,), float(rank + 1)), "db_gate": None, "dw_down": None, "dw_up": None}
    for _ in range(2):
        order.forward(x, {})
        order.backward(x, x, {}, G)
    out[rank] = dict(log=log, violations=violations, counts=order.rk.counts_all.tolist(), dw_gate=float(G["dw_gate"][0]))
    dist.barrier()
    dist.destroy_process_group()


def test_expert_parallel_phase_order_and_barriers_with_two_ranks():
    """EpStepOrder (what EpProcessRank runs) over two gloo ranks with stub phase calls: the order of the calls, a
    barrier in front of every phase that reads what peers wrote, the count all-gather between route and dispatch, and
    the shared-gradient reduction at the end of the backward."""
    world, port = 2, 31500 + os.getpid() % 1000
    manager = mp.Manager()
    out = manager.dict()
    mp.spawn(_order_worker, args=(world, port, out), nprocs=world, join=True)
    step = ["route", "gather", "dispatch", "|", "experts", "|", "combine",
            "|", "backward_combine", "|", "backward_experts", "|", "backward_dispatch", "reduce"]
    for r_ in range(world):
        assert out[r_]["log"] == step + step
        assert out[r_]["violations"] == []                      # no phase ran before its inputs existed on every rank
        assert out[r_]["counts"] == [[1, 1, 1, 1], [2, 2, 2, 2]]
        assert out[r_]["dw_gate"] == 6.0                          # (1 + 2) after the first step's reduction, doubled by the second
