"""Out-of-order readiness under real concurrency: a producer thread puts shuffled chunks on its
own stream while consumer threads poll td_get on theirs.  Several outcomes are valid, so the
checks are the invariants every outcome must satisfy, plus bit parity of every batch's payload,
cu_seqlens and advantages with what the oracle gathers for the same indices."""
import threading
import time

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import td_oracle as ora
from paper_2507_19017_b200 import binding as td
from paper_2507_19017_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2507_19017_b200 import build
    build.build()
    from tests import gpu_helpers
    return gpu_helpers


def run_concurrent(G, w, consumer_threads):
    """consumer_threads: list of consumer numbers, one polling thread each (a consumer may
    appear several times: ranks that share one controller)."""
    g = G.GpuDock(w)
    puts = [op for op in w.ops if op.kind == "put"]
    batches = [[] for _ in consumer_threads]
    errors = []
    done_putting = threading.Event()
    served = {c: 0 for c in set(consumer_threads)}
    lock = threading.Lock()

    def producer():
        try:
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                for op in puts:
                    g.put_op(op, stream=s)
                s.synchronize()
        except Exception as e:       # pragma: no cover
            errors.append(e)
        finally:
            done_putting.set()

    def consumer(slot, c):
        try:
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                pc, rc = g.token_caps(w.micro_batch)
                bufs = td.GetBuffers(g.dock, c, w.micro_batch, prompt_tokens_cap=pc, response_tokens_cap=rc)
                idle = 0
                deadline = time.time() + 120
                while True:
                    assert time.time() < deadline, "consumer did not finish in time"
                    g.dock.get(bufs, stream=s)
                    b = g.read(bufs, stream=s)
                    assert b.status == 0
                    if b.n_samples:
                        batches[slot].append(b)
                        with lock:
                            served[c] += b.n_samples
                        idle = 0
                    else:
                        with lock:
                            finished = served[c] >= w.n
                        if finished:
                            break
                        if done_putting.is_set():
                            idle += 1
                            assert idle < 2000, "dock is full but the consumer cannot drain it"
        except Exception as e:
            errors.append(e)

    threads = [threading.Thread(target=producer)]
    threads += [threading.Thread(target=consumer, args=(i, c)) for i, c in enumerate(consumer_threads)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=150)
    assert not any(t.is_alive() for t in threads), "a thread did not finish"
    if errors:
        raise errors[0]
    torch.cuda.synchronize()
    return g, batches


def check_outcome(G, w, g, consumer_threads, batches):
    # the oracle holds the same data (any put order gives the same rows back)
    o = H.make_oracle(w)
    idx = np.arange(w.n, dtype=np.int32)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, idx)
        o.put(c, idx, cu, data)
    per_consumer = {}
    partial = 0
    for slot, c in enumerate(consumer_threads):
        for b in batches[slot]:
            assert b.n_samples % w.N == 0 and 0 < b.n_samples <= w.micro_batch
            assert np.all(np.diff(b.indices) > 0)
            grp = b.indices.reshape(-1, w.N)
            assert np.all(grp[:, 0] % w.N == 0) and np.array_equal(grp, grp[:, :1] + np.arange(w.N))
            want = o.gather(c, b.indices)
            want.status = b.status
            G.assert_batch_equal(b, want, f"consumer {c} thread {slot}")
            per_consumer.setdefault(c, []).extend(b.indices.tolist())
            partial += b.n_samples < w.micro_batch
    for c, got in per_consumer.items():
        assert len(got) == w.n and sorted(got) == list(range(w.n)), f"consumer {c}: not exactly once"
        assert H.popcount_words(g.table(5, c, np.uint32)) == w.n
        assert H.popcount_words(g.table(4, c, np.uint32)) == w.G
    st = g.dock.status()
    assert st.error_word == 0
    for c in per_consumer:
        assert st.got_samples[c] == w.n
    return partial, st


def test_concurrent_producer_and_four_consumers_small(G):
    w = wl.make_custom("conc", 128, 4, 8, prompt_len=(8, 200), response=("lognormal", 300.0, 0.4, 1200),
                       vocab=32000, micro_batch=32, seed=41, schedule="interleaved", chunk=(1, 24), poll_every=8)
    g, batches = run_concurrent(G, w, [0, 1, 2, 3])
    check_outcome(G, w, g, [0, 1, 2, 3], batches)


def test_two_threads_share_one_controller(G):
    """Two polling threads for consumer 0 (and two for the advantage consumer): the claim by
    atomicOr must hand every group to exactly one of them."""
    w = wl.make_custom("share", 256, 2, 4, prompt_len=(4, 60), response=("uniform", 4, 200), vocab=32000,
                       micro_batch=16, seed=42, schedule="interleaved", chunk=(1, 64), poll_every=8)
    threads = [0, 0, 3, 3, 1]
    g, batches = run_concurrent(G, w, threads)
    partial, st = check_outcome(G, w, g, threads, batches)
    assert all(len(b) > 0 for b in batches)


def test_config4_concurrent_full_size(G):
    w = wl.make_config(4)
    g, batches = run_concurrent(G, w, [0, 1, 2, 3])
    partial, st = check_outcome(G, w, g, [0, 1, 2, 3], batches)


def test_concurrent_cascade_with_write_backs(G):
    """The whole sample flow with every party on its own stream and thread: a producer puts the
    id columns in shuffled chunks, three inference states poll, and send their column back for
    each batch they are served (td_put_back, batch size read on the device), the actor update
    polls for what has become complete.  Checked like the other concurrent runs: exactly once per
    consumer, and every batch equal to what the oracle gathers for its indices once it holds
    the same rows."""
    w = wl.make_custom("conc-cascade", 96, 4, 8, prompt_len=(8, 200), response=("lognormal", 300.0, 0.4, 1200),
                       vocab=32000, micro_batch=32, seed=45, schedule="cascade", chunk=(4, 40), poll_every=4,
                       with_entropy=True)
    g = G.GpuDock(w)
    puts = [op for op in w.ops if op.kind == "put"]
    produces = {}
    for op in w.ops:
        if op.kind == "put_back":
            produces[op.consumer] = op.columns
    workers = sorted(produces)
    updater = [c for c in range(len(w.consumers)) if c not in produces][0]
    pool_dev = {c: G.to_device(a, g.device) for c, a in w.pool.items()}
    errors, lock = [], threading.Lock()
    batches = {c: [] for c in range(len(w.consumers))}

    def producer():
        try:
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                for op in puts:
                    g.put_op(op, stream=s)
                s.synchronize()
        except Exception as e:       # pragma: no cover
            errors.append(e)

    def party(c):
        try:
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                pc, rc = g.token_caps(w.micro_batch)
                bufs = td.GetBuffers(g.dock, c, w.micro_batch, prompt_tokens_cap=pc, response_tokens_cap=rc)
                served, deadline = 0, time.time() + 120
                while served < w.n:
                    assert time.time() < deadline, f"consumer {c} did not finish in time"
                    g.dock.get(bufs, stream=s)
                    if c in produces:                      # enqueued before the host knows the batch size
                        g.dock.put_back(bufs, [(col, pool_dev[col]) for col in produces[c]], stream=s)
                    b = g.read(bufs, stream=s)
                    assert b.status == 0
                    if b.n_samples:
                        batches[c].append(b)
                        served += b.n_samples
        except Exception as e:
            errors.append(e)

    threads = [threading.Thread(target=producer)] + [threading.Thread(target=party, args=(c,))
                                                     for c in range(len(w.consumers))]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=150)
    assert not any(t.is_alive() for t in threads), "a thread did not finish"
    if errors:
        raise errors[0]
    torch.cuda.synchronize()

    # the oracle is given the same rows: the ids, then every write-back as the workers made it
    o = H.make_oracle(w)
    idx = np.arange(w.n, dtype=np.int32)
    for name in ("prompt_ids", "response_ids"):
        c = w.column_index(name)
        cu, data = w.pack(c, idx)
        o.put(c, idx, cu, data)
    for c in workers:
        for b in batches[c]:
            H.oracle_put_back(w, o, b, produces[c])
    for c in range(len(w.consumers)):
        got = []
        for b in batches[c]:
            assert b.n_samples % w.N == 0 and np.all(np.diff(b.indices) > 0)
            want = o.gather(c, b.indices)
            want.status = b.status
            G.assert_batch_equal(b, want, f"consumer {c}")
            got.extend(b.indices.tolist())
        assert sorted(got) == list(range(w.n)), f"consumer {c}: not exactly once"
    st = g.dock.status()
    assert st.error_word == 0
    for col in w.pool:
        assert st.put_accepted[col] == w.n
    full = (1 << len(w.columns)) - 1
    assert np.all(g.table(0, 0, np.uint32) == full)           # every column of every sample stored
