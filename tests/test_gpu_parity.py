"""Parity of the CUDA library with the CPU oracle on the same seeded inputs, through the C ABI.
Indices, offsets, bitmaps, cu_seqlens and payload are compared bit for bit; the fp32 advantages
within 1e-6 relative / 1e-7 absolute (both sides accumulate in double)."""
import dataclasses

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


# ------------------------------------------------------------------ the five shapes
def test_config1_tiny_random_order(G):
    w = wl.make_config(1)
    g, o, batches = G.replay_both(w, check_state_every=5)
    assert sum(b.n_samples for _, b in batches) == w.n * len(w.consumers)


def test_config1_padded(G):
    w = wl.make_config(1)
    G.replay_both(w, mode=td.PADDED)


@pytest.mark.parametrize("cid", [2, 3])
def test_bulk_configs_full_size(G, cid):
    w = wl.make_config(cid)
    g, o, batches = G.replay_both(w)
    assert sum(b.n_samples for _, b in batches) == w.n * len(w.consumers)


def test_config5_full_size_packed(G):
    w = wl.make_config(5)
    g, o, batches = G.replay_both(w)
    assert sum(b.n_samples for _, b in batches) == w.n * len(w.consumers)


def test_config5_full_size_padded_drain(G):
    """The R1-shaped dock drained to exhaustion into right-padded rows for an id-only consumer and
    for the actor update (one set of output buffers per consumer, reused get after get): every
    batch and the final tables against the oracle."""
    w = wl.make_config(5, schedule="none")
    o, g = H.make_oracle(w), G.GpuDock(w)
    idx = np.arange(w.n, dtype=np.int32)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, idx)
        o.put(c, idx, cu, data); g.put(c, idx, cu, data)
    served = {0: 0, 3: 0}
    for j in range(w.n // w.micro_batch + 1):                   # one get past the end: an empty batch
        for cons in (0, 3):
            want = o.get(cons, w.micro_batch, ora.PADDED, w.pad_prompt_to, w.pad_response_to)
            got = g.get(cons, w.micro_batch, td.PADDED, w.pad_prompt_to, w.pad_response_to)
            G.assert_batch_equal(got, want, f"padded get {j} consumer {cons}")
            served[cons] += got.n_samples
    assert served == {0: w.n, 3: w.n}
    G.assert_state_equal(g, o, arenas=False, ctx="padded drain")
    G.assert_stats_equal(g, o, "padded drain")


def test_config4_interleaved_serialized(G):
    """The out-of-order schedule executed in order on one stream is deterministic: bit-exact."""
    w = wl.make_config(4)
    g, o, batches = G.replay_both(w, check_state_every=400, arenas=False)
    per = {c: 0 for c in range(len(w.consumers))}
    partial = 0
    for c, b in batches:
        per[c] += b.n_samples
        partial += b.n_samples < w.micro_batch
    assert all(v == w.n for v in per.values())
    assert partial > 100          # the schedule really met partially ready docks


# --------------------------------------------------------------- shapes that stress the kernels
def test_cascade_write_back_small(G):
    """Generation puts, the inference states send their columns back for the batches they were
    served (batch size read on the device, no host round trip), the actor update takes what is
    complete: every get and the final state against the oracle."""
    w = wl.make_custom("cascade-small", 24, 4, 3, prompt_len=(5, 70), response=("uniform", 1, 300),
                       vocab=50000, micro_batch=8, seed=31, schedule="cascade", chunk=(1, 12),
                       poll_every=3, with_entropy=True)
    g, o, batches = G.replay_both(w, check_state_every=7)
    upd = len(w.consumers) - 1
    assert sum(b.n_samples for c, b in batches if c == upd) == w.n


def test_cascade_batched_polls(G):
    """The same flow with one td_get_many and one td_put_back_many per poll."""
    w = wl.make_custom("cascade-batched", 24, 4, 3, prompt_len=(5, 70), response=("uniform", 1, 300),
                       vocab=50000, micro_batch=8, seed=33, schedule="cascade_batched", chunk=(1, 12),
                       poll_every=3, with_entropy=True)
    g, o, batches = G.replay_both(w, check_state_every=5)
    upd = len(w.consumers) - 1
    assert sum(b.n_samples for c, b in batches if c == upd) == w.n
    w2 = wl.make_config(2, schedule="cascade_batched")
    g, o, batches = G.replay_both(w2)
    assert sum(b.n_samples for c, b in batches if c == upd) == w2.n


def test_cascade_replayed_from_a_cuda_graph(G):
    """Nothing in the flow needs the host (batch sizes are read on the device), so a whole
    iteration - reset, generation puts, gets, write-backs - can be recorded once and replayed:
    every get of the replay against the oracle, twice."""
    import torch
    w = wl.make_custom("cascade-graph", 16, 4, 2, prompt_len=(5, 70), response=("uniform", 1, 300),
                       vocab=50000, micro_batch=8, seed=35, schedule="cascade_batched", chunk=(4, 12),
                       poll_every=2)
    o = H.make_oracle(w)
    want = H.replay_oracle(w, o)
    g = G.GpuDock(w)
    pool_dev = {c: G.to_device(a, g.device) for c, a in w.pool.items()}
    calls, bufs_of_get, last = [], [], {}
    for j, op in enumerate(w.ops):
        if op.kind == "put":
            cu, data = w.pack(op.column, op.indices)
            calls.append(("put", op.column, G.to_device(np.ascontiguousarray(op.indices, np.int32), g.device),
                          G.to_device(cu, g.device), G.to_device(data, g.device)))
        elif op.kind == "get_many":
            bufs = [g.buffers(c, op.max_samples, key=("graph", j)) for c in op.group]      # one set per get
            calls.append(("get_many", g.dock.plan(bufs)))
            for c, b in zip(op.group, bufs):
                last[c] = b
                bufs_of_get.append((c, b))
        else:
            calls.append(("back_many", [(last[c], col, pool_dev[col]) for c, col in op.group]))

    def run():
        g.dock.reset()
        for call in calls:
            if call[0] == "put":
                g.dock.put(call[1], call[2], call[3], call[4])
            elif call[0] == "get_many":
                g.dock.get_many(call[1])
            else:
                g.dock.put_back_many(call[1])

    run()                                   # eager once (also the first use of every kernel)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        run()
    for rep in range(2):
        for _c, b in bufs_of_get:           # stale results must not pass for fresh ones
            b.result.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert len(bufs_of_get) == len(want)
        for k, ((c, b), (wc, wb)) in enumerate(zip(bufs_of_get, want)):
            assert c == wc
            G.assert_batch_equal(g.read(b), wb, f"replay {rep} get {k} consumer {c}")
        G.assert_state_equal(g, o, ctx=f"replay {rep}")


@pytest.mark.parametrize("cid", [2, 3])
def test_cascade_write_back_full_size(G, cid):
    base = wl.make_config(cid, schedule="none")
    w = wl.make_custom(f"cascade-{cid}", base.G, base.N, base.S,
                       prompt_len=(128, 1024) if cid == 2 else (256, 2048),
                       response=("lognormal", 1500.0 if cid == 2 else 3000.0, 0.25, 4096 if cid == 2 else 16384),
                       vocab=152064, micro_batch=base.micro_batch, seed=wl.BASE_SEED + 100 + cid,
                       schedule="cascade", chunk=(16, 256), poll_every=6, with_entropy=cid == 3)
    g, o, batches = G.replay_both(w, check_state_every=0, arenas=cid == 2)
    upd = len(w.consumers) - 1
    assert sum(b.n_samples for c, b in batches if c == upd) == w.n


@pytest.mark.parametrize("N,Gp,S", [(1, 12, 3), (3, 10, 5), (5, 8, 2), (7, 6, 1), (32, 4, 4), (33, 3, 3)])
def test_group_sizes_that_do_not_divide_a_warp(G, N, Gp, S):
    w = wl.make_custom("odd", Gp, N, S, prompt_len=(1, 70), response=("uniform", 0, 200), vocab=50000,
                       micro_batch=2 * N, seed=100 + N, with_entropy=True, schedule="random_order", chunk=(1, 9))
    G.replay_both(w, check_state_every=7)
    G.replay_both(w, mode=td.PADDED)


def test_all_row_alignments_and_lengths(G):
    """Row lengths 0..70 in every order: every source/destination misalignment of the 16-byte
    copy path, for 4-byte and 2-byte elements, heads and tails included."""
    w = wl.make_custom("align", 64, 2, 4, prompt_len=(0, 37), response=("uniform", 0, 70), vocab=1 << 20,
                       micro_batch=6, seed=11, with_entropy=True, schedule="random_order", chunk=(1, 7))
    G.replay_both(w)
    w2 = wl.make_custom("align2", 64, 2, 4, prompt_len=(0, 37), response=("uniform", 0, 70), vocab=1 << 20,
                        micro_batch=128, seed=12, with_entropy=True, schedule="bulk")
    G.replay_both(w2)


def test_source_buffer_edges_are_not_overread(G):
    """Put from, and get into, tensors that sit at odd element offsets inside guard regions:
    the guards must stay untouched and the payload exact."""
    w = wl.make_custom("edge", 8, 2, 2, prompt_len=(1, 50), response=("uniform", 1, 300), vocab=1000,
                       micro_batch=16, seed=5, with_entropy=True, schedule="none")
    o = H.make_oracle(w)
    g = G.GpuDock(w)
    idx = np.arange(w.n, dtype=np.int32)
    for c, spec in enumerate(w.columns):
        cu, data = w.pack(c, idx)
        o.put(c, idx, cu, data)
        dev = G.to_device(data, g.device)
        guard = torch.full((dev.numel() + 64,), -1 if dev.dtype != torch.bfloat16 else 1.0, dtype=dev.dtype, device=g.device)
        shift = 3 if spec.cls != wl.SCALAR else 1
        guard[shift:shift + dev.numel()] = dev
        view = guard[shift:shift + dev.numel()]
        g.dock.put(c, G.to_device(idx, g.device), G.to_device(cu, g.device) if cu is not None else None, view)
    torch.cuda.synchronize()
    want = o.get(3, w.n)
    bufs = g.buffers(3, w.n)
    # exact-size outputs embedded in guard buffers
    embedded = {}
    for c, t in list(bufs.cols.items()):
        need = want.columns[c].size
        big = torch.zeros(need + 48, dtype=t.dtype, device=g.device)
        fill = torch.full_like(big, 7)
        big.copy_(fill)
        shift = 5
        bufs.cols[c] = big[shift:shift + need]
        bufs.caps[c] = need
        bufs.struct.col[c] = bufs.cols[c].data_ptr()
        bufs.struct.col_capacity_elems[c] = need
        embedded[c] = (big, shift, need)
    g.dock.get(bufs)
    got = g.read(bufs)
    G.assert_batch_equal(got, want, "edge")
    for c, (big, shift, need) in embedded.items():
        host = G.to_host(big)
        ref = G.to_host(torch.full((1,), 7, dtype=big.dtype))[0]
        assert np.all(host[:shift] == ref) and np.all(host[shift + need:] == ref), f"guard of column {c}"


def test_many_tiles_look_back(G):
    """More groups than one scan tile holds (256), random readiness, several consumers and
    batch sizes: ranks must come from the look-back chain across tiles."""
    w = wl.make_custom("tiles", 3000, 1, 8, prompt_len=(0, 4), response=("uniform", 0, 6), vocab=100,
                       micro_batch=700, seed=21, schedule="interleaved", chunk=(1, 900), poll_every=3)
    g, o, batches = G.replay_both(w, arenas=False)
    assert max(b.n_groups for _, b in batches) > 256
    w2 = wl.make_custom("tiles2", 1100, 2, 4, prompt_len=(0, 4), response=("uniform", 0, 6), vocab=100,
                        micro_batch=2200, seed=22, schedule="bulk")
    g, o, batches = G.replay_both(w2)
    assert batches[0][1].n_samples == 2200


def test_wide_tiles_of_a_large_dock(G):
    """More than 65536 groups: scan tiles take four passes of 256 groups each.  Random partial
    readiness, gets of thousands of groups and of a few, ranks across passes and tiles."""
    w = wl.make_custom("wide", 70000, 1, 4, prompt_len=(0, 2), response=("uniform", 0, 3), vocab=100,
                       micro_batch=9000, seed=23, schedule="interleaved", chunk=(1, 30000), poll_every=3)
    g, o, batches = G.replay_both(w, arenas=False)
    assert max(b.n_groups for _, b in batches) > 4096
    w2 = wl.make_custom("wide2", 66048, 2, 8, prompt_len=(0, 2), response=("uniform", 0, 3), vocab=100,
                        micro_batch=64, seed=24, schedule="none")
    o2, g2 = H.make_oracle(w2), G.GpuDock(w2)
    idx = np.arange(w2.n, dtype=np.int32)[::-1].copy()          # every sample, highest first
    for c in range(len(w2.columns)):
        cu, data = w2.pack(c, idx)
        o2.put(c, idx, cu, data); g2.put(c, idx, cu, data)
    for c in (0, 3, 0, 3):
        G.assert_batch_equal(g2.get(c, 64), o2.get(c, 64), f"wide2 consumer {c}")
    G.assert_state_equal(g2, o2, arenas=False, ctx="wide2")


def _twelve_tile_dock(G):
    w = wl.make_custom("timeout", 12 * 256, 1, 4, prompt_len=(0, 3), response=("uniform", 0, 5), vocab=100,
                       micro_batch=12 * 256, seed=31, schedule="none")
    o, g = H.make_oracle(w), G.GpuDock(w)
    idx = np.arange(w.n, dtype=np.int32)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, idx)
        o.put(c, idx, cu, data); g.put(c, idx, cu, data)
    return w, o, g


def _claimed(g, consumer):
    return H.popcount_words(g.table(4, consumer, np.uint32))


@pytest.mark.parametrize("skip_tile", [5, 0, 11])
def test_lookback_wait_that_runs_out_serves_nothing_and_hands_claims_back(G, skip_tile):
    """A scan tile that never publishes its descriptor: the tiles behind it wait their (short)
    limit and give up, the get reports TD_ERR_LOOKBACK_TIMEOUT and serves nothing - and the
    groups that the tiles ahead of it had already claimed are free again, so that the next get
    serves the lowest groups as if nothing had happened."""
    w, o, g = _twelve_tile_dock(G)
    one = g.get(2, 256)                                          # an ordinary get first: groups 0..255 to consumer 2
    G.assert_batch_equal(one, o.get(2, 256), "before")
    before = {c: _claimed(g, c) for c in range(len(w.consumers))}
    g.dock.debug_lookback(poll_limit=64, skip_tile=skip_tile)
    for cons, m in ((3, w.n), (2, 1024)):
        got = g.get(cons, m)
        assert got.status == td.ERR_LOOKBACK_TIMEOUT and got.n_samples == 0 and got.n_groups == 0
        assert got.prompt_tokens == 0 and got.response_tokens == 0
    assert {c: _claimed(g, c) for c in range(len(w.consumers))} == before
    rep = g.dock.validate()
    assert rep.violations == 0 and rep.served[2] == 256 and rep.served[3] == 0
    st = g.dock.status()
    assert st.error_word == td.ERR_LOOKBACK_TIMEOUT and st.n_lookback_timeouts >= 2
    assert st.got_samples[3] == 0 and st.got_samples[2] == 256
    g.dock.debug_lookback()                                      # default limit, no tile withheld
    for cons, m in ((3, 700), (2, 1024), (3, w.n), (2, w.n)):
        G.assert_batch_equal(g.get(cons, m), o.get(cons, m), f"after, consumer {cons}")
    G.assert_state_equal(g, o, arenas=False, ctx="after timeouts")
    assert _claimed(g, 3) == w.G and _claimed(g, 2) == w.G


def test_lookback_timeout_inside_a_plan(G):
    """td_get_many over a scan that does not come through: every request of every consumer returns
    nothing, no claim stays behind, and the same plan serves everything once the scan works."""
    w, o, g = _twelve_tile_dock(G)
    bufs = [g.buffers(c, 800, key=j) for j, c in enumerate((0, 3, 0, 3, 1))]
    plan = g.dock.plan(bufs)
    g.dock.debug_lookback(poll_limit=64, skip_tile=3)
    g.dock.get_many(plan)
    for b in bufs:
        r = g.read(b)
        assert r.status == td.ERR_LOOKBACK_TIMEOUT and r.n_samples == 0
    assert all(_claimed(g, c) == 0 for c in range(len(w.consumers)))
    assert g.dock.validate().violations == 0
    g.dock.debug_lookback()
    g.dock.get_many(plan)
    for b, c in zip(bufs, (0, 3, 0, 3, 1)):
        G.assert_batch_equal(g.read(b), o.get(c, 800), f"plan consumer {c}")
    G.assert_state_equal(g, o, arenas=False, ctx="plan after timeout")


def test_scan_scratch_in_use_by_a_later_launch_is_refused(G):
    """A ticket word that carries a later launch's sequence number (what a tile finds when two
    gets in flight were given the same scratch): the scan refuses, nothing is served or claimed,
    and the scratch is usable again for the next get."""
    w, o, g = _twelve_tile_dock(G)
    bufs = g.buffers(0, 1024)
    ticket = bufs.scratch[:8].view(torch.int64)
    ticket.fill_(-(1 << 32))                                     # sequence number 0xffffffff, no tile started
    g.dock.debug_lookback(poll_limit=64)
    g.dock.get(bufs)
    r = g.read(bufs)
    assert r.status == td.ERR_LOOKBACK_TIMEOUT and r.n_samples == 0
    assert _claimed(g, 0) == 0 and g.dock.validate().violations == 0
    g.dock.debug_lookback()
    g.dock.get(bufs)
    G.assert_batch_equal(g.read(bufs), o.get(0, 1024), "after the refusal")


# ------------------------------------------------------------------- batched calls
def _many_vs_serial(G, w, mode=td.PACKED, fused=False):
    """All columns in one td_put_many, all gets of the schedule in one td_get_many; the oracle
    runs the same calls one by one."""
    o = H.make_oracle(w)
    g = G.GpuDock(w)
    pad_p, pad_r = (w.pad_prompt_to, w.pad_response_to) if mode == td.PADDED else (0, 0)
    items, keep = [], []
    for op in w.ops:
        if op.kind == "put":
            cu, data = w.pack(op.column, op.indices)
            o.put(op.column, op.indices, cu, data)
            t = (op.column, G.to_device(np.ascontiguousarray(op.indices, np.int32), g.device),
                 G.to_device(cu, g.device) if cu is not None else None, G.to_device(data, g.device))
            items.append(t)
    g.dock.put_many(items)
    G.assert_state_equal(g, o, ctx="after put_many")
    gets = [op for op in w.ops if op.kind == "get"]
    # fused: the actor update's requests ask for the token stream, the other consumers' do not
    kws = [G.stream_args(w, op.consumer) if fused and w.consumers[op.consumer].advantage else {} for op in gets]
    bufs = [g.buffers(op.consumer, op.max_samples, mode, pad_p, pad_r, key=j, **kws[j]) for j, op in enumerate(gets)]
    plan = g.dock.plan(bufs)
    g.dock.get_many(plan)
    for j, op in enumerate(gets):
        want = o.get(op.consumer, op.max_samples, mode, pad_p, pad_r, **kws[j])
        G.assert_batch_equal(g.read(bufs[j]), want, f"request {j}")
    G.assert_state_equal(g, o, ctx="after get_many")
    G.assert_stats_equal(g, o, "many")
    # the same plan again: everything is consumed, every request comes back empty
    g.dock.get_many(plan)
    assert all(g.read(b).n_samples == 0 for b in bufs)
    return g, o, plan, bufs


def test_put_many_get_many_small(G):
    w = wl.make_custom("many", 24, 3, 4, prompt_len=(1, 70), response=("uniform", 0, 200), vocab=50000,
                       micro_batch=9, seed=31, with_entropy=True, schedule="bulk")
    _many_vs_serial(G, w)
    _many_vs_serial(G, w, mode=td.PADDED)


@pytest.mark.parametrize("cid", [2, 3, 5])
def test_put_many_get_many_full_size(G, cid):
    _many_vs_serial(G, wl.make_config(cid))


def test_one_request_for_the_whole_batch(G):
    """A consumer that asks for everything at once: thousands of rows in one request (the large
    finalize block, scalar elements spread over many chunks), alone and inside a plan."""
    w = wl.make_config(2, schedule="none")
    o = H.make_oracle(w)
    g = G.GpuDock(w)
    idx = np.arange(w.n, dtype=np.int32)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, idx)
        o.put(c, idx, cu, data); g.put(c, idx, cu, data)
    upd = len(w.consumers) - 1
    kw = G.stream_args(w, upd)
    G.assert_batch_equal(g.get(upd, w.n, **kw), o.get(upd, w.n, **kw), "whole batch, td_get")
    bufs = [g.buffers(c, w.n, key="plan") for c in range(upd)]
    plan = g.dock.plan(bufs)
    g.dock.get_many(plan)
    for c in range(upd):
        G.assert_batch_equal(g.read(bufs[c]), o.get(c, w.n), f"whole batch, plan, consumer {c}")
    G.assert_state_equal(g, o, ctx="whole batch")


# ------------------------------------------------------------------- fused token stream
def test_fused_stream_every_alignment(G):
    """prompt row followed by response row at cu_seq, for every consumer, lengths 0..70 in every
    order (zero-length prompts and responses included), packed and padded columns beside it."""
    w = wl.make_custom("fuse", 64, 2, 4, prompt_len=(0, 37), response=("uniform", 0, 70), vocab=1 << 20,
                       micro_batch=6, seed=41, with_entropy=True, schedule="random_order", chunk=(1, 7))
    G.replay_both(w, fused=True)
    G.replay_both(w, mode=td.PADDED, fused=True)
    w2 = wl.make_custom("fuse2", 9, 7, 3, prompt_len=(1, 300), response=("uniform", 0, 5000), vocab=1 << 20,
                        micro_batch=63, seed=42, schedule="bulk")
    G.replay_both(w2, fused=True)


def test_fused_stream_in_a_plan(G):
    w = wl.make_custom("fuse3", 24, 3, 4, prompt_len=(1, 70), response=("uniform", 0, 200), vocab=50000,
                       micro_batch=9, seed=43, with_entropy=True, schedule="bulk")
    _many_vs_serial(G, w, fused=True)
    _many_vs_serial(G, w, mode=td.PADDED, fused=True)


@pytest.mark.parametrize("cid", [2, 3])
def test_fused_stream_full_size(G, cid):
    _many_vs_serial(G, wl.make_config(cid), fused=True)


# ------------------------------------------------------------------- left-padded prompts
def _put_everything(w, o, g):
    idx = np.arange(w.n, dtype=np.int32)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, idx)
        o.put(c, idx, cu, data); g.put(c, idx, cu, data)


def test_left_padded_prompts_every_alignment(G):
    """TD_OUT_LEFT_PAD_PROMPT: prompt rows flush with the end of their width.  Lengths 0..37 (rows
    of no length and rows that fill the width included) at widths whose rows start on every
    4-byte phase, drained in small gets, in one get of everything and through a plan; the fused
    stream beside it is unchanged by the flag."""
    w = wl.make_custom("lpad", 64, 2, 4, prompt_len=(0, 37), response=("uniform", 0, 70), vocab=1 << 20,
                       micro_batch=6, seed=13, with_entropy=True, schedule="none")
    # a 2-byte prompt column beside the ids, and pad patterns that are not zero
    pads = {"prompt_ids": 0xDEADBEEF, "response_ids": 0x7FC00001, "entropy": 0xABCD}
    w.columns = [dataclasses.replace(c, pad_bits=pads.get(c.name, 0)) for c in w.columns]
    w.columns.append(wl.ColumnSpec("prompt_weight", "bf16", wl.PROMPT, 0x3F80))
    w.data["prompt_weight"] = np.random.Generator(np.random.PCG64(5)).integers(
        0, 1 << 16, size=int(w.len_prompt.sum()), dtype=np.uint16)
    w.consumers = wl.standard_consumers(w.columns)
    upd = len(w.consumers) - 1
    for widths in ((37, 70), (38, 71), (39, 73), (40, 72)):
        o, g = H.make_oracle(w), G.GpuDock(w)
        _put_everything(w, o, g)
        kw = G.stream_args(w, upd)
        for j in range(w.n // 6 + 1):
            for cons, extra in ((0, {}), (upd, kw)):
                want = o.get(cons, 6, ora.PADDED, *widths, out_flags=ora.OUT_LEFT_PAD_PROMPT, **extra)
                got = g.get(cons, 6, td.PADDED, *widths, left_pad=True, **extra)
                G.assert_batch_equal(got, want, f"widths {widths} get {j} consumer {cons}")
        # everything at once for another consumer, and two more consumers through one plan
        G.assert_batch_equal(g.get(1, w.n, td.PADDED, *widths, left_pad=True),
                             o.get(1, w.n, ora.PADDED, *widths, out_flags=ora.OUT_LEFT_PAD_PROMPT), "whole batch")
        bufs = [g.buffers(2, 20, td.PADDED, *widths, key=f"plan{q}", left_pad=True) for q in range(3)]
        g.dock.get_many(g.dock.plan(bufs))
        for q in range(3):
            G.assert_batch_equal(g.read(bufs[q]), o.get(2, 20, ora.PADDED, *widths, out_flags=ora.OUT_LEFT_PAD_PROMPT),
                                 f"plan request {q}")
        G.assert_state_equal(g, o, ctx=f"left-padded, widths {widths}")
    # rows right-padded when the flag is absent, on the same buffers' shapes; unknown flags refused
    G.assert_batch_equal(g.get(2, 20, td.PADDED, 40, 72), o.get(2, 20, ora.PADDED, 40, 72), "flag absent")
    bad = g.buffers(2, 20, td.PADDED, 40, 72, key="bad flags")
    bad.struct.flags = 2
    with pytest.raises(td.TdError):
        g.dock.get(bad)


def test_left_padded_prompts_long_rows(G):
    """Rows of many pipeline stages, widths far beyond the longest row, chunk borders inside pad
    and payload alike: the 7B-shaped dock's prompts and responses, 64-sample gets."""
    w = wl.make_config(2, schedule="none")
    o, g = H.make_oracle(w), G.GpuDock(w)
    _put_everything(w, o, g)
    upd = len(w.consumers) - 1
    for j in range(3):
        for cons in (0, upd):
            want = o.get(cons, 64, ora.PADDED, w.pad_prompt_to + 3, w.pad_response_to, out_flags=ora.OUT_LEFT_PAD_PROMPT)
            got = g.get(cons, 64, td.PADDED, w.pad_prompt_to + 3, w.pad_response_to, left_pad=True)
            G.assert_batch_equal(got, want, f"get {j} consumer {cons}")
            # independent of the oracle: a prompt row ends with its tokens, the pad fills the front
            c0 = w.column_index("prompt_ids")
            assert H.bits_equal(got.columns[c0], H.expected_padded(w, c0, got.indices, w.pad_prompt_to + 3, left=True))


def test_fused_stream_of_a_float_pair_and_truncation(G):
    """Any prompt/response pair of one element size can be fused; a stream buffer that is too
    small ends the batch before the first group that does not fit and leaves it available."""
    w = wl.make_custom("fuse4", 8, 2, 2, prompt_len=(3, 30), response=("uniform", 1, 60), vocab=500,
                       micro_batch=16, seed=44, schedule="none")
    o = H.make_oracle(w)
    g = G.GpuDock(w)
    idx = np.arange(w.n, dtype=np.int32)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, idx)
        o.put(c, idx, cu, data); g.put(c, idx, cu, data)
    upd = len(w.consumers) - 1
    pair = (w.column_index("prompt_ids"), w.column_index("old_logprob"))
    room = int((w.len_prompt + w.len_response)[:6].sum()) + 5          # three groups and a bit
    want = o.get(upd, 16, seq=pair, seq_adv=True, seq_cap=room)
    got = g.get(upd, 16, seq=pair, seq_adv=True, seq_cap=room)
    assert want.n_groups == 3 and want.status & td.ERR_OUT_TRUNCATED
    G.assert_batch_equal(got, want, "truncated stream")
    G.assert_batch_equal(g.get(upd, 16, seq=pair, seq_adv=True, key="rest"),
                         o.get(upd, 16, seq=pair, seq_adv=True), "the rest")
    G.assert_state_equal(g, o, ctx="fuse4")
    # host-side refusals: classes swapped, element sizes differ, advantage twin without advantages
    bad = g.buffers(0, 16, seq=(pair[1], pair[0]), key="bad")
    with pytest.raises(td.TdError):
        g.dock.get(bad)
    bad2 = g.buffers(0, 16, seq_adv=True, key="bad2")
    with pytest.raises(td.TdError):
        g.dock.get(bad2)


def test_get_many_partial_readiness_and_reuse(G):
    """A plan that asks for more than is ready: early requests are filled, later ones come back
    short or empty; after more puts the same plan serves the rest."""
    w = wl.make_custom("many2", 20, 2, 2, prompt_len=(1, 30), response=("uniform", 1, 60), vocab=500,
                       micro_batch=8, seed=32, schedule="bulk")
    o = H.make_oracle(w)
    g = G.GpuDock(w)
    first = np.arange(0, 22, dtype=np.int32)          # 11 groups
    rest = np.arange(22, w.n, dtype=np.int32)
    for idx in (first,):
        for c in range(len(w.columns)):
            cu, data = w.pack(c, idx)
            o.put(c, idx, cu, data); g.put(c, idx, cu, data)
    gets = [op for op in w.ops if op.kind == "get"]
    bufs = [g.buffers(op.consumer, op.max_samples, key=j) for j, op in enumerate(gets)]
    plan = g.dock.plan(bufs)
    g.dock.get_many(plan)
    served = 0
    for j, op in enumerate(gets):
        want = o.get(op.consumer, op.max_samples)
        G.assert_batch_equal(g.read(bufs[j]), want, f"first call, request {j}")
        served += want.n_samples
    assert served == 22 * len(w.consumers)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, rest)
        o.put(c, rest, cu, data); g.put(c, rest, cu, data)
    g.dock.get_many(plan)
    for j, op in enumerate(gets):
        G.assert_batch_equal(g.read(bufs[j]), o.get(op.consumer, op.max_samples), f"second call, request {j}")
    G.assert_state_equal(g, o, ctx="many2")


def test_put_many_same_column_twice_and_errors(G):
    w = wl.make_custom("many3", 8, 2, 2, prompt_len=(1, 30), response=("uniform", 1, 60), vocab=500,
                       micro_batch=8, seed=33, schedule="none")
    o = H.make_oracle(w)
    g = G.GpuDock(w)
    rid = w.column_index("response_ids")
    a, b = np.array([0, 1, 2, 3], np.int32), np.array([3, 4, 5, 99], np.int32)
    items = []
    for idx in (a, b):
        cu, data = w.pack(rid, np.clip(idx, 0, w.n - 1))
        o.put(rid, idx, cu, data)
        items.append((rid, G.to_device(idx, g.device), G.to_device(cu, g.device), G.to_device(data, g.device)))
    g.dock.put_many(items)
    G.assert_state_equal(g, o, ctx="same column twice")
    G.assert_stats_equal(g, o, "same column twice")


# ----------------------------------------------------------------------------- error paths
def test_put_errors_are_counted_and_skipped(G):
    w = wl.make_custom("err", 8, 4, 2, prompt_len=(3, 40), response=("uniform", 1, 90), vocab=1000,
                       micro_batch=8, seed=7, schedule="none")
    o = H.make_oracle(w)
    g = G.GpuDock(w)
    rid, old, rew = w.column_index("response_ids"), w.column_index("old_logprob"), w.column_index("reward")

    def both(col, idx, cu, data):
        idx = np.asarray(idx, np.int32)
        o.put(col, idx, cu, data)
        g.put(col, idx, cu, data)

    both(rid, [0, 1, 2], *w.pack(rid, np.array([0, 1, 2], np.int32)))
    both(rid, [1, -1, w.n, 3], *w.pack(rid, np.array([1, 0, 0, 3], np.int32)))       # dup, 2 x oob, ok
    bad_cu = np.array([0, int(w.len_response[0]) + 1], np.int32)
    both(old, [0], bad_cu, np.zeros(bad_cu[1], np.float32))                           # length mismatch
    both(rid, [5], np.array([4, 2], np.int32), np.zeros(8, np.int32))                 # decreasing cu
    both(rew, [0, 0 + w.n, 1], None, np.array([1.0, 2.0, 3.0], np.float32))           # scalar oob
    both(rew, [1, 2], None, np.array([9.0, 4.0], np.float32))                         # scalar dup
    G.assert_state_equal(g, o, ctx="errors")
    G.assert_stats_equal(g, o, "errors")
    st = g.dock.status()
    assert st.error_word == td.ERR_OOB_INDEX | td.ERR_DUP_PUT | td.ERR_LEN_MISMATCH | td.ERR_BAD_LENGTH


def test_bad_cu_entry_in_the_middle_of_a_put_skips_only_that_row(G):
    """cu arrays that go down in the middle of a many-row put, by a little and by more than any
    row is long (row positions can then not be searched): only the offending rows are refused,
    every other row of the call is stored with its payload, and later puts are not disturbed."""
    w = wl.make_custom("badcu", 40, 4, 4, prompt_len=(3, 900), response=("uniform", 1, 3000), vocab=50000,
                       micro_batch=160, seed=12, with_entropy=True, schedule="none")
    room = 2 * w.shard_capacity(wl.RESPONSE)                    # the misread rows come out longer than the true ones
    o, g = H.make_oracle(w, response_cap=room), G.GpuDock(w, response_cap=room)
    rid, pid, ent = w.column_index("response_ids"), w.column_index("prompt_ids"), w.column_index("entropy")
    idx = np.arange(w.n, dtype=np.int32)

    def both(col, ind, cu, data):
        o.put(col, ind, cu, data); g.put(col, ind, cu, data)

    # response ids: one entry far below its predecessor (row 50 then ends before it starts, and row
    # 51 reaches back over it), another one two elements below (row 100)
    cu, data = w.pack(rid, idx)
    bad = cu.copy()
    bad[51] = cu[50] - 2000
    bad[101] = cu[100] - 2
    both(rid, idx, bad, data)
    assert o.stats().n_bad_length == 2 and o.stats().put_accepted[rid] == w.n - 2
    # prompt ids of the second half with a last entry of -1: the array's total is useless, every
    # row but the last is in order
    half = idx[w.n // 2:]
    cu_p, data_p = w.pack(pid, half)
    cu_p2 = cu_p.copy()
    cu_p2[-1] = -1
    both(pid, half, cu_p2, data_p)
    assert o.stats().n_bad_length == 3 and o.stats().put_accepted[pid] == len(half) - 1
    # clean puts afterwards (the dock has seen irregular arrays; results must not change); the
    # entropy rows of the two samples whose response length was misread are refused
    both(pid, idx[:w.n // 2], *w.pack(pid, idx[:w.n // 2]))
    both(ent, idx, *w.pack(ent, idx))
    assert o.stats().n_len_mismatch == 2
    G.assert_state_equal(g, o, ctx="bad cu")
    G.assert_stats_equal(g, o, "bad cu")
    assert g.dock.status().error_word == td.ERR_BAD_LENGTH | td.ERR_LEN_MISMATCH
    # what was stored can be served: the id-only consumers get every complete group
    for cons in (0, 1):
        G.assert_batch_equal(g.get(cons, w.n), o.get(cons, w.n), f"consumer {cons}")


def test_same_sample_twice_in_one_call_is_safe(G):
    """The same index more than once inside one put is outside what the dock specifies (which copy
    stays is open), but it must be safe: the row ends up stored once, the tables stay sound, the
    counters agree with the tables, and - both copies being equal here - the row reads back."""
    w = wl.make_custom("twice", 6, 4, 2, prompt_len=(3, 40), response=("uniform", 5000, 9000), vocab=1000,
                       micro_batch=24, seed=17, schedule="none")
    g = G.GpuDock(w)
    rid, pid, rew = w.column_index("response_ids"), w.column_index("prompt_ids"), w.column_index("reward")
    order = np.array([0, 1, 1, 2, 3, 3, 3] + list(range(4, w.n)) + [w.n - 1], np.int32)     # long rows: several chunks each
    for c in (rid, pid, rew, w.column_index("old_logprob"), w.column_index("ref_logprob")):
        cu, data = w.pack(c, order)
        g.put(c, order, cu, data)
    rep = g.dock.validate()
    assert rep.violations == 0
    assert list(rep.stored[:len(w.columns)]) == [w.n] * len(w.columns)
    st = g.dock.status()
    assert all(st.put_accepted[c] == w.n for c in range(len(w.columns)))
    assert st.error_word & ~td.ERR_DUP_PUT == 0
    got = g.get(3, w.n)
    assert got.n_samples == w.n and got.status == 0
    for c, spec in enumerate(w.columns):
        assert H.bits_equal(got.columns[c], w.data[spec.name]), spec.name


def test_arena_full_refuses_only_rows_without_room(G):
    w = wl.make_custom("full", 4, 4, 2, prompt_len=(10, 10), response=("uniform", 5, 60), vocab=1000,
                       micro_batch=16, seed=9, schedule="none")
    room =(w.len_response.reshape(2, -1).astype(np.int64) + 7) // 8 * 8
    cap = int(room.sum(axis=1).min() // 2 // 8 * 8)            # about half of what a shard needs
    o = H.make_oracle(w, response_cap=cap)
    g = G.GpuDock(w, response_cap=cap)
    rid = w.column_index("response_ids")
    order = np.random.default_rng(1).permutation(w.n).astype(np.int32)
    cu, data = w.pack(rid, order)
    accepted = o.put(rid, order, cu, data)
    g.put(rid, order, cu, data)
    assert 0 < accepted < w.n
    G.assert_state_equal(g, o, ctx="arena full")
    G.assert_stats_equal(g, o, "arena full")
    assert g.dock.status().error_word == td.ERR_ARENA_FULL


def test_one_put_of_many_passes_in_random_order(G):
    """One call carrying 9000 rows in shuffled order over 12 shards: several allocation passes,
    warps whose rows fall into different shards, and - with a tight arena - an overflow that
    only shows up in a late pass.  Offsets must still be those of a walk in call order."""
    w = wl.make_custom("passes", 3000, 3, 12, prompt_len=(0, 9), response=("uniform", 0, 40), vocab=999,
                       micro_batch=9000, seed=61, with_entropy=True, schedule="none")
    order = np.random.default_rng(3).permutation(w.n).astype(np.int32)
    for tight in (False, True):
        room = (w.len_response.reshape(w.S, -1).astype(np.int64) + 7) // 8 * 8
        cap = int(room.sum(axis=1).min() * 0.9 // 8 * 8) if tight else None
        o = H.make_oracle(w, response_cap=cap)
        g = G.GpuDock(w, response_cap=cap)
        for c in (w.column_index("response_ids"), w.column_index("prompt_ids"), w.column_index("entropy")):
            cu, data = w.pack(c, order)
            o.put(c, order, cu, data)
            g.put(c, order, cu, data)
        G.assert_state_equal(g, o, ctx=f"tight={tight}")
        G.assert_stats_equal(g, o, f"tight={tight}")
        assert (o.stats().n_arena_full > 0) == tight


def test_output_capacity_truncation_matches(G):
    w = wl.make_custom("trunc", 8, 2, 2, prompt_len=(3, 40), response=("uniform", 1, 90), vocab=1000,
                       micro_batch=16, seed=7, schedule="none")
    o = H.make_oracle(w)
    g = G.GpuDock(w)
    idx = np.arange(w.n, dtype=np.int32)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, idx)
        o.put(c, idx, cu, data); g.put(c, idx, cu, data)
    rid = w.column_index("response_ids")
    room = int(w.len_response[:6].sum()) + 1
    caps = {rid: room, w.column_index("prompt_ids"): int(w.len_prompt.sum())}
    want = o.get(0, w.n, capacities=caps)
    got = g.get(0, w.n, capacities=caps)
    assert want.status == ora.ERR_OUT_TRUNC and want.n_samples == 6
    G.assert_batch_equal(got, want, "truncated")
    G.assert_state_equal(g, o, ctx="after truncation")
    G.assert_batch_equal(g.get(0, w.n), o.get(0, w.n), "rest")
    # padded: a row longer than the width ends the batch before its group
    wide = int(w.len_response.max())
    want = o.get(1, w.n, ora.PADDED, 40, wide - 1)
    got = g.get(1, w.n, td.PADDED, 40, wide - 1)
    G.assert_batch_equal(got, want, "padded truncation")
    G.assert_stats_equal(g, o, "truncation")


def _host_batch(G, g, bufs, host) -> "object":
    """What td_get_host / td_get_many_host left in the pinned host mirrors, as a Batch."""
    from oracle import td_oracle as ora
    r = host.result
    b = ora.Batch()
    b.n_samples, b.n_groups, b.status = r.n_samples, r.n_groups, r.status
    b.prompt_tokens, b.response_tokens = r.prompt_tokens, r.response_tokens
    k = b.n_samples
    b.indices = host.indices[:k].numpy().copy()
    b.cu_prompt, b.cu_response = host.cu_prompt[:k + 1].numpy().copy(), host.cu_response[:k + 1].numpy().copy()
    b.cu_seq = host.cu_seq[:k + 1].numpy().copy()
    for c, t in host.cols.items():
        cls = g.dock.columns[c][1]
        tot = k if cls == td.SCALAR else (b.prompt_tokens if cls == td.PROMPT else b.response_tokens)
        b.columns[c] = G.to_host(t[:tot])
    if host.advantages is not None:
        b.advantages = host.advantages[:k].numpy().copy()
    return b


def test_host_buffer_calls_single_and_batched(G):
    """Host tensors in, host tensors out: td_put_host + td_get_host per call, and
    td_put_many_host + td_get_many_host for a whole step, against the oracle."""
    import torch
    w = wl.make_custom("host", 24, 3, 4, prompt_len=(1, 70), response=("uniform", 0, 200), vocab=50000,
                       micro_batch=9, seed=51, with_entropy=True, schedule="bulk")
    gets = [op for op in w.ops if op.kind == "get"]

    def pinned(a):
        t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else np.ascontiguousarray(a))
        return (t.view(torch.bfloat16) if a.dtype == np.uint16 else t).pin_memory()

    for batched in (False, True, "staged", "in place"):
        o = H.make_oracle(w)
        g = G.GpuDock(w)
        items = []
        for op in w.ops:
            if op.kind == "put":
                cu, data = w.pack(op.column, op.indices)
                o.put(op.column, op.indices, cu, data)
                items.append((op.column, pinned(np.ascontiguousarray(op.indices, np.int32)),
                              pinned(cu) if cu is not None else None, pinned(data)))
        need = [g.dock.put_host_stage_bytes(c, i.numel(), d.numel()) for c, i, _cu, d in items]
        bufs = [g.buffers(op.consumer, op.max_samples, key=("host", j)) for j, op in enumerate(gets)]
        if batched == "in place":         # payload buffers in pinned host memory, written by the gather itself
            pc, rc = g.token_caps(w.micro_batch)
            bufs = [td.GetBuffers(g.dock, op.consumer, op.max_samples, prompt_tokens_cap=pc, response_tokens_cap=rc,
                                  host_payload=True) for op in gets]
            for b in bufs:
                for t in b.cols.values():
                    t.view(torch.uint8).fill_(0xA5)
        hosts = [td.HostGetBuffers(b) for b in bufs]
        if batched:
            stage = torch.empty(sum(need), dtype=torch.uint8, device=g.device)
            g.dock.put_many_host(items, stage)
            plan = g.dock.plan(bufs)
            meta = None
            if batched in ("staged", "in place"):   # results, indices, cu_seqlens and advantages of all requests in one transfer
                meta = torch.empty(g.dock.get_many_host_stage_bytes(plan), dtype=torch.uint8, device=g.device)
            g.dock.get_many_host(plan, hosts, meta)
        else:
            stage = torch.empty(max(need), dtype=torch.uint8, device=g.device)
            for c, i, cu, d in items:
                g.dock.put_host(c, i, cu, d, stage)
                torch.cuda.synchronize()          # one staging buffer: free again before the next put
            for b, h in zip(bufs, hosts):
                g.dock.get_host(b, h)
        for j, op in enumerate(gets):
            want = o.get(op.consumer, op.max_samples)
            G.assert_batch_equal(_host_batch(G, g, bufs[j], hosts[j]), want, f"batched={batched} request {j}")
        G.assert_state_equal(g, o, ctx=f"host batched={batched}")


@pytest.mark.parametrize("in_place", [False, True])
def test_two_waves_with_host_buffers_on_two_streams(G, in_place):
    """The columns every worker state needs are put first; the states that need nothing else are
    served on a second stream behind that put while the other columns are still being put on the
    first; the actor update follows the second put.  Every batch is the oracle's: which samples
    an id-only state is served, and what it is handed, does not depend on the columns still in
    flight."""
    import torch
    w = wl.make_custom("waves", 48, 4, 4, prompt_len=(1, 300), response=("uniform", 0, 3000), vocab=50000,
                       micro_batch=32, seed=53, with_entropy=True, schedule="bulk")
    gets = [op for op in w.ops if op.kind == "get"]

    def pinned(a):
        t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else np.ascontiguousarray(a))
        return (t.view(torch.bfloat16) if a.dtype == np.uint16 else t).pin_memory()

    o, g = H.make_oracle(w), G.GpuDock(w)
    first = {w.column_index("prompt_ids"), w.column_index("response_ids")}
    upd = len(w.consumers) - 1
    items = {True: [], False: []}
    for op in w.ops:
        if op.kind == "put":
            cu, data = w.pack(op.column, op.indices)
            o.put(op.column, op.indices, cu, data)
            items[op.column in first].append((op.column, pinned(np.ascontiguousarray(op.indices, np.int32)),
                                              pinned(cu) if cu is not None else None, pinned(data)))
    pc, rc = g.token_caps(w.micro_batch)
    bufs = [td.GetBuffers(g.dock, op.consumer, op.max_samples, prompt_tokens_cap=pc, response_tokens_cap=rc,
                          host_payload=in_place) for op in gets]
    hosts = [td.HostGetBuffers(b) for b in bufs]
    waves = []
    for early in (True, False):
        sel = [j for j, op in enumerate(gets) if (op.consumer != upd) == early]
        plan = g.dock.plan([bufs[j] for j in sel])
        stage = torch.empty(sum(g.dock.put_host_stage_bytes(c, i.numel(), d.numel()) for c, i, _cu, d in items[early]),
                            dtype=torch.uint8, device=g.device)
        meta = torch.empty(g.dock.get_many_host_stage_bytes(plan), dtype=torch.uint8, device=g.device)
        waves.append((items[early], stage, plan, [hosts[j] for j in sel], meta))
    side = torch.cuda.Stream()
    ev = torch.cuda.Event()
    for rep in range(3):                       # the buffers, plans and staging areas are reused step after step
        if rep:
            g.dock.reset(); o.reset()
            for op in w.ops:
                if op.kind == "put":
                    o.put(op.column, op.indices, *w.pack(op.column, op.indices))
        (it_a, st_a, plan_a, hosts_a, meta_a), (it_b, st_b, plan_b, hosts_b, meta_b) = waves
        g.dock.put_many_host(it_a, st_a)
        ev.record()
        g.dock.put_many_host(it_b, st_b)
        side.wait_event(ev)
        g.dock.get_many_host(plan_a, hosts_a, meta_a, stream=side)
        g.dock.get_many_host(plan_b, hosts_b, meta_b)
        for j, op in enumerate(gets):
            want = o.get(op.consumer, op.max_samples)
            G.assert_batch_equal(_host_batch(G, g, bufs[j], hosts[j]), want, f"step {rep} request {j}")
        G.assert_state_equal(g, o, ctx=f"two waves, step {rep}")
        G.assert_stats_equal(g, o, f"two waves, step {rep}")


def test_validate_reports_planted_damage(G):
    """td_debug_validate passes on a dock in use and names damage planted into its tables from
    the host side (an unknown status bit, two rows at one place, a served mark without a claim)."""
    import torch
    w = wl.make_custom("validate", 8, 2, 2, prompt_len=(3, 30), response=("uniform", 1, 60), vocab=500,
                       micro_batch=4, seed=61, schedule="bulk")
    g, o, _ = G.replay_both(w)
    rep = g.dock.validate()
    assert rep.violations == 0
    assert list(rep.stored[:len(w.columns)]) == [w.n] * len(w.columns)
    assert list(rep.served[:len(w.consumers)]) == [w.n] * len(w.consumers)
    used = int(((w.len_response.astype(np.int64) + 7) // 8 * 8).sum())
    assert rep.arena_elems_used[2] == used
    status = g.dock.table(0).view(torch.int32)
    status[3] |= 1 << 20
    assert g.dock.validate().violations & td.BAD_STATUS_BITS
    status[3] &= ~(1 << 20)
    off = g.dock.table(2, 2).view(torch.int64)
    keep = off[1].item()
    off[1] = off[0]
    assert g.dock.validate().violations & td.BAD_ROW_OVERLAP
    off[1] = keep
    claim = g.dock.table(4, 1).view(torch.int32)
    claim[0] &= ~1
    assert g.dock.validate().violations & td.BAD_SERVED_UNCLAIMED
    claim[0] |= 1
    assert g.dock.validate().violations == 0


def test_host_argument_checks(G):
    w = wl.make_config(1)
    g = G.GpuDock(w)
    bufs = g.buffers(0, 8)
    with pytest.raises(td.TdError):
        g.dock.get(bufs, max_samples=3)             # fewer than one group
    idx = torch.zeros(4, dtype=torch.int32, device=g.device)
    with pytest.raises(td.TdError):
        g.dock.put(1, idx, None, idx)               # ragged column without cu
    with pytest.raises(td.TdError):
        g.dock.put(99, idx, idx, idx)
    small = td.GetBuffers(g.dock, 0, 8, prompt_tokens_cap=8, response_tokens_cap=8)
    small.struct.scratch_bytes = 8
    with pytest.raises(td.TdError) as e:
        g.dock.get(small)
    assert e.value.code == td.EWORKSPACE


def test_reset_and_reuse(G):
    w = wl.make_config(1)
    g, o, _ = G.replay_both(w)
    g.dock.reset(); o.reset()
    G.assert_state_equal(g, o, arenas=False, ctx="after reset")
    assert g.get(0, 8).n_samples == 0
    for op in w.ops:
        if op.kind == "put":
            cu, data = w.pack(op.column, op.indices)
            o.put(op.column, op.indices, cu, data); g.put(op.column, op.indices, cu, data)
    G.assert_batch_equal(g.get(3, w.n), o.get(3, w.n), "after reuse")


def test_zero_variance_groups_give_exact_zero(G):
    w = wl.make_custom("zv", 6, 5, 1, prompt_len=(1, 4), response=("uniform", 1, 4), vocab=10,
                       micro_batch=30, seed=2, schedule="none")
    w.data["reward"][:5] = np.float32(0.3)
    w.data["reward"][5:10] = np.array([0, 1, 1, 0, 1], np.float32)
    w.data["reward"][10:15] = np.float32(1e4) + np.float32(1e-3) * np.arange(5, dtype=np.float32)
    w.ops = wl._bulk_ops(w)
    g, o, batches = G.replay_both(w)
    adv = [b for c, b in batches if c == 3][0].advantages
    assert np.all(adv[:5] == 0.0)
