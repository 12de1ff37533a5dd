"""td_get_static: the get for callers that cannot hand over scratch memory (code that runs where
device memory may not be allocated: a frozen memory pool, a plug-in that owns only its input
and output buffers).  Its scan scratch is a fixed array inside the library, so its answers must
be those of td_get, call after call, although that array still holds the previous call's
contents.  Collected last on purpose: a run that stops at the first failure has then already
run every other test."""
import ctypes as C

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2507_19017_b200 import binding as td
from paper_2507_19017_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2507_19017_b200 import build
    build.build()
    from tests import gpu_helpers
    return gpu_helpers


def filled_dock(G, w):
    g = G.GpuDock(w)
    idx = np.arange(w.n, dtype=np.int32)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, idx)
        g.put(c, idx, cu, data)
    return g


def test_static_scratch_get_matches_td_get_on_consecutive_calls(G):
    # 2000 prompts: more than one launch's finalize kernel can scan by itself, so every call runs
    # the scan kernel (8 tiles: ticket, tile descriptors, start ranks and candidate list all live
    # in the shared array) on top of whatever the call before it left there
    from tests import helpers as H
    w = wl.make_custom("noalloc", 2000, 2, 4, prompt_len=(1, 40), response=("uniform", 0, 90), vocab=30000,
                       micro_batch=500, seed=77, with_entropy=True, schedule="none")
    ref, sta = filled_dock(G, w), filled_dock(G, w)
    ora_dock = H.make_oracle(w)
    idx = np.arange(w.n, dtype=np.int32)
    for c in range(len(w.columns)):
        ora_dock.put(c, idx, *w.pack(c, idx))
    launches = sta.dock.launch_count()
    calls = [(3, 500), (0, 500), (3, 500), (3, 64), (0, 2 * w.n), (1, 10), (1, 10), (3, 1500)]
    for j, (consumer, m) in enumerate(calls):
        want = ref.get(consumer, m, key=j)                    # td_get with caller-supplied scratch
        bufs = sta.buffers(consumer, m, key=j)
        bufs.struct.scratch, bufs.struct.scratch_bytes = None, 0          # nothing to lean on
        sta.dock.get_static(bufs)
        got = sta.read(bufs)
        G.assert_batch_equal(got, want, f"call {j}")
        G.assert_batch_equal(got, ora_dock.get(consumer, m), f"call {j} against the oracle")
        assert got.status == 0
    assert sta.dock.launch_count() - launches == 3 * len(calls)           # select, finalize, gather every time
    assert ref.get(3, 4000, key="x").n_samples == w.n - 2564  # the drains stayed in step to the end
    b = sta.buffers(3, 4000, key="x")
    sta.dock.get_static(b)
    assert sta.read(b).n_samples == w.n - 2564
    for c in range(len(w.consumers)):
        assert np.array_equal(sta.table(4, c, np.uint32), ref.table(4, c, np.uint32))
        assert np.array_equal(sta.table(5, c, np.uint32), ref.table(5, c, np.uint32))
    assert sta.dock.status().error_word == 0


def test_static_scratch_get_refuses_docks_beyond_its_limit(G):
    cols = [("i32", "prompt", 0), ("f32", "scalar", 0)]
    big = td.Dock(16385, 1, 1, cols, [(3, 3, False)], 8, 8, 1)
    bufs = td.GetBuffers(big, 0, 4, prompt_tokens_cap=16, response_tokens_cap=16)
    before = big.launch_count()
    with pytest.raises(td.TdError) as e:
        big.get_static(bufs)
    assert e.value.code == td.ETOOLARGE
    assert big.launch_count() == before                       # nothing was enqueued
    assert b"prompts" in td.lib().td_strerror(td.ETOOLARGE)
    big.get(bufs)                                             # the ordinary get still serves it
    torch.cuda.synchronize()
    assert bufs.read_result().n_samples == 0
    ok = td.Dock(16384, 1, 1, cols, [(3, 3, False)], 8, 8, 1)
    bufs2 = td.GetBuffers(ok, 0, 4, prompt_tokens_cap=16, response_tokens_cap=16)
    ok.get_static(bufs2)
    torch.cuda.synchronize()
    assert bufs2.read_result().n_samples == 0 and bufs2.read_result().status == 0
