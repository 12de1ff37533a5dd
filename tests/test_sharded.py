"""One dock sharded over ranks (warehouse j on rank j mod P): the routing of puts, the metadata
broadcast, the replica-driven selection and the assembly of a batch on the worker state's home
rank.  Two gloo ranks on the CPU, each with its own local dock, are checked batch by batch
against ONE unsharded dock that is given the same calls: same samples, same order, same bits,
every sample exactly once per consumer.  The ranks' local docks here are CPU docks behind the
adapter seam of sharded.py; on a GPU the same code drives the CUDA library (last test)."""
import os
import socket
import sys

import numpy as np
import pytest

torch = pytest.importorskip("torch")

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2507_19017_b200 import sharded as sh
from paper_2507_19017_b200 import workloads as wl
from tests import helpers as H


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _t(a: np.ndarray) -> torch.Tensor:
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    return torch.from_numpy(a)


def _n(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).numpy().view(np.uint16)
    return t.contiguous().numpy()


class CpuLocal:
    """A rank's own dock for the CPU tests: the plain C dock the tests use as their oracle, put
    behind the interface sharded.py expects of a local dock."""

    def __init__(self, smap, rank, w, prompt_cap, response_cap):
        from oracle import td_oracle as ora
        g_local, s_local = smap.local_shape(rank)
        self.o = ora.OracleDock(g_local, smap.N, s_local, w.column_tuples(), w.consumer_tuples(), prompt_cap,
                                response_cap, w.column_index("reward"), 1e-6)
        self.device = torch.device("cpu")
        self.G = g_local

    def put(self, column, indices, cu, data):
        self.o.put(column, _n(indices), _n(cu) if cu is not None else None, _n(data))

    def get(self, consumer, max_samples):
        b = self.o.get(consumer, max_samples)
        assert b.status == 0
        return sh.LocalBatch(b.n_samples, _t(b.indices), _t(b.cu_prompt), _t(b.cu_response),
                             {c: _t(a) for c, a in b.columns.items()},
                             _t(b.advantages) if b.advantages is not None else None)

    def status_words(self):
        return _t(self.o.status().view(np.int32))

    def claim_bits(self, consumer):
        return _t(H.bit_list(self.o.claim_words(consumer), self.G))

    def reset(self):
        self.o.reset()


def make_workload():
    return wl.make_custom("sharded", 24, 3, 6, prompt_len=(1, 30), response=("uniform", 0, 70), vocab=5000,
                          micro_batch=12, seed=91, with_entropy=True, schedule="interleaved", chunk=(1, 9), poll_every=5)


def assert_same_batch(got: sh.ShardedBatch, want, ctx):
    assert got.n_samples == want.n_samples and got.n_groups == want.n_groups, ctx
    assert np.array_equal(_n(got.indices), want.indices), ctx
    assert np.array_equal(_n(got.cu_prompt), want.cu_prompt) and np.array_equal(_n(got.cu_response), want.cu_response), ctx
    assert np.array_equal(_n(got.cu_seq), want.cu_seq), ctx
    assert (got.prompt_tokens, got.response_tokens) == (want.prompt_tokens, want.response_tokens), ctx
    assert sorted(got.columns) == sorted(want.columns), ctx
    for c in want.columns:
        assert H.bits_equal(_n(got.columns[c]), want.columns[c]), f"{ctx} column {c}"
    if want.advantages is None:
        assert got.advantages is None
    else:
        assert np.allclose(_n(got.advantages), want.advantages, rtol=1e-6, atol=1e-7), ctx
        assert np.array_equal(_n(got.advantages) == 0, want.advantages == 0), ctx


def run_schedule(w, dock, reference, rank, world, collect):
    """The workload's calls on the sharded dock (put j is made by rank j mod world, the others
    hand in nothing; every poll is preceded by the metadata broadcast) and on the unsharded
    reference; every batch that arrives on this rank is compared at once."""
    served = {c: [] for c in range(len(w.consumers))}
    n_put = n_get = 0
    dirty = False
    for op in w.ops:
        if op.kind == "put":
            cu, data = w.pack(op.column, op.indices)
            reference.put(op.column, op.indices, cu, data)
            mine = n_put % world == rank
            k = len(op.indices) if mine else 0
            dock.put(op.column, _t(np.ascontiguousarray(op.indices[:k], np.int32)),
                     _t(cu[:k + 1]) if cu is not None else None,
                     _t(data[:int(cu[k]) if cu is not None else k]))
            n_put += 1
            dirty = True
        else:
            if dirty:
                dock.sync()
                dirty = False
            want = reference.get(op.consumer, op.max_samples)
            got = dock.get(op.consumer, op.max_samples)
            home = dock.home_of(op.consumer)
            assert (got is not None) == (rank == home)
            if got is not None:
                assert_same_batch(got, want, f"get {n_get} consumer {op.consumer}")
                collect.append((op.consumer, got.n_samples))
            served[op.consumer].extend(want.indices.tolist())
            n_get += 1
    for c, idx in served.items():
        assert sorted(idx) == list(range(w.n)), f"consumer {c}: not exactly once"
    return n_get


def _rank_main(rank, world, port):
    import torch.distributed as dist
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        w = make_workload()
        smap = sh.ShardMap(w.G, w.N, w.S, world)
        cap_p, cap_r = w.shard_capacity(wl.PROMPT), w.shard_capacity(wl.RESPONSE)
        local = CpuLocal(smap, rank, w, cap_p, cap_r)
        dock = sh.ShardedDock(smap, local, sh.Comm(), w.column_tuples(), w.consumer_tuples())
        reference = H.make_oracle(w)
        got = []
        n_get = run_schedule(w, dock, reference, rank, world, got)
        # this rank is home to every other consumer: it received exactly their batches
        assert {c for c, _ in got} <= {c for c in range(len(w.consumers)) if c % world == rank}
        assert sum(n for _, n in got) == w.n * len([c for c in range(len(w.consumers)) if c % world == rank])
        assert n_get > 20
        # the local docks together hold every sample once: each rank's share is its warehouses'
        assert H.popcount_words(local.o.consumed_words(0)) == smap.local_shape(rank)[0] * w.N
        # a reset empties the replica too; the dock is usable again
        dock.reset(); reference.reset()
        dock.sync()
        empty = dock.get(0, 12)
        assert (empty is None) == (rank != dock.home_of(0)) and (empty is None or empty.n_samples == 0)
    finally:
        dist.barrier()
        dist.destroy_process_group()


def test_shard_map_is_a_bijection_and_keeps_order():
    for G, N, S, P in ((24, 3, 6, 2), (40, 2, 8, 3), (16, 4, 4, 4), (12, 1, 12, 5)):
        m = sh.ShardMap(G, N, S, P)
        seen = []
        for r in range(P):
            glob = m.global_samples_of(r)
            g_local, s_local = m.local_shape(r)
            assert len(glob) == g_local * N and s_local == len(m.shards_of(r))
            assert torch.equal(m.local_sample(glob), torch.arange(len(glob)))          # round trip
            assert torch.all(m.owner_of_group(glob // N) == r)
            assert torch.all(glob[1:] > glob[:-1])                                     # local order keeps global order
            assert sorted(set((glob // N // m.gps).tolist())) == m.shards_of(r)        # whole warehouses
            seen.extend(glob.tolist())
        assert sorted(seen) == list(range(G * N))
    with pytest.raises(ValueError):
        sh.ShardMap(10, 2, 4, 2)            # S does not divide G
    with pytest.raises(ValueError):
        sh.ShardMap(8, 2, 2, 4)             # fewer warehouses than ranks


def test_one_rank_is_the_plain_dock():
    """P = 1: every exchange is a local copy; the batches are the unsharded dock's."""
    w = make_workload()
    smap = sh.ShardMap(w.G, w.N, w.S, 1)
    local = CpuLocal(smap, 0, w, w.shard_capacity(wl.PROMPT), w.shard_capacity(wl.RESPONSE))
    dock = sh.ShardedDock(smap, local, sh.Comm(), w.column_tuples(), w.consumer_tuples())
    got = []
    assert run_schedule(w, dock, H.make_oracle(w), 0, 1, got) > 20
    assert sum(n for _, n in got) == w.n * len(w.consumers)
    with pytest.raises(ValueError):
        dock.put(1, torch.tensor([0], dtype=torch.int32), torch.tensor([3, 1], dtype=torch.int32),
                 torch.zeros(4, dtype=torch.int32))


def test_two_gloo_ranks_serve_what_one_dock_serves():
    import torch.multiprocessing as mp
    mp.spawn(_rank_main, args=(2, _free_port()), nprocs=2, join=True)


def test_four_gloo_ranks_with_uneven_warehouse_counts():
    """Six warehouses over four ranks: two ranks hold two, two hold one."""
    import torch.multiprocessing as mp
    mp.spawn(_rank_main, args=(4, _free_port()), nprocs=4, join=True)


@pytest.mark.gpu
def test_one_rank_on_the_gpu_goes_through_the_same_code():
    """The sharded dock with one rank whose local dock is the CUDA library: same schedule, every
    batch bit for bit the unsharded oracle's."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2507_19017_b200 import build
    build.build()
    w = make_workload()
    smap = sh.ShardMap(w.G, w.N, w.S, 1)
    local = sh.CudaLocal(smap, 0, w.column_tuples(), w.consumer_tuples(), w.shard_capacity(wl.PROMPT),
                         w.shard_capacity(wl.RESPONSE), w.column_index("reward"),
                         int(w.len_prompt.max()), int(w.len_response.max()))
    dock = sh.ShardedDock(smap, local, sh.Comm(), w.column_tuples(), w.consumer_tuples())

    class OnDevice:
        """run_schedule hands in CPU tensors; the CUDA dock wants them on its device."""
        def __init__(self, d):
            self.d = d
        def put(self, column, idx, cu, data):
            dev = self.d.device
            self.d.put(column, idx.to(dev), cu.to(dev) if cu is not None else None, data.to(dev))
        def sync(self):
            self.d.sync()
        def home_of(self, c):
            return self.d.home_of(c)
        def get(self, c, m):
            b = self.d.get(c, m)
            cpu = lambda t: t.cpu() if t is not None else None
            return sh.ShardedBatch(b.n_samples, b.n_groups, cpu(b.indices), cpu(b.cu_prompt), cpu(b.cu_response),
                                   cpu(b.cu_seq), {c_: t.cpu() for c_, t in b.columns.items()}, cpu(b.advantages),
                                   b.prompt_tokens, b.response_tokens)

    got = []
    assert run_schedule(w, OnDevice(dock), H.make_oracle(w), 0, 1, got) > 20
    assert sum(n for _, n in got) == w.n * len(w.consumers)
    assert local.dock.status().error_word == 0 and local.dock.validate().violations == 0
