"""GPU-side test glue: drive the CUDA library through its binding and bring results back as
numpy arrays shaped like the oracle wrapper's Batch, so the two can be compared field by field."""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import numpy as np
import torch

from oracle import td_oracle as ora
from paper_2507_19017_b200 import binding as td
from paper_2507_19017_b200 import workloads as wl
from tests import helpers as H

REL_TOL, ABS_TOL = 1e-6, 1e-7      # advantages; everything else is compared bit for bit


def to_device(a: np.ndarray, device) -> torch.Tensor:
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def to_host(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


class GpuDock:
    def __init__(self, w: wl.Workload, prompt_cap=None, response_cap=None, eps: float = 1e-6):
        self.w = w
        self.dock = td.Dock(w.G, w.N, w.S, w.column_tuples(), w.consumer_tuples(),
                            prompt_cap if prompt_cap is not None else w.shard_capacity(wl.PROMPT),
                            response_cap if response_cap is not None else w.shard_capacity(wl.RESPONSE),
                            w.column_index("reward"), eps)
        self.device = self.dock.device
        self._bufs: Dict = {}
        self._keep = []

    # -- calls ------------------------------------------------------------
    def put(self, column: int, indices, cu, data, stream=None):
        idx = to_device(np.ascontiguousarray(indices, dtype=np.int32), self.device)
        cut = to_device(np.ascontiguousarray(cu, dtype=np.int32), self.device) if cu is not None else None
        dat = to_device(data, self.device)
        if dat.numel() == 0:
            dat = torch.zeros(8, dtype=dat.dtype, device=self.device)[:0]
        self.dock.put(column, idx, cut, dat, stream)
        self._keep.append((idx, cut, dat))
        if len(self._keep) > 64:
            torch.cuda.synchronize()
            self._keep.clear()

    def put_op(self, op: wl.Op, stream=None):
        cu, data = self.w.pack(op.column, op.indices)
        self.put(op.column, op.indices, cu, data, stream)

    def token_caps(self, max_samples: int):
        p = int(np.sort(self.w.len_prompt)[::-1][:max_samples].sum(dtype=np.int64))
        r = int(np.sort(self.w.len_response)[::-1][:max_samples].sum(dtype=np.int64))
        return p, r

    def buffers(self, consumer: int, max_samples: int, mode: int = td.PACKED, pad_p: int = 0,
                pad_r: int = 0, capacities=None, want=None, key=None, seq=None, seq_adv=False,
                seq_cap=None, left_pad=False) -> td.GetBuffers:
        k = (consumer, max_samples, mode, pad_p, pad_r, key,
             tuple(sorted(capacities.items())) if capacities else None, tuple(want) if want else None,
             seq, seq_adv, seq_cap, left_pad)
        if k not in self._bufs:
            pc, rc = self.token_caps(max_samples)
            self._bufs[k] = td.GetBuffers(self.dock, consumer, max_samples, mode, pad_p, pad_r,
                                          capacities, want, pc, rc, seq, seq_adv, seq_cap,
                                          left_pad_prompts=left_pad)
        return self._bufs[k]

    def get(self, consumer: int, max_samples: int, mode: int = td.PACKED, pad_p: int = 0, pad_r: int = 0,
            capacities=None, want=None, stream=None, key=None, seq=None, seq_adv=False,
            seq_cap=None, left_pad=False) -> ora.Batch:
        bufs = self.buffers(consumer, max_samples, mode, pad_p, pad_r, capacities, want, key, seq, seq_adv, seq_cap,
                            left_pad)
        self.dock.get(bufs, stream)
        return self.read(bufs, stream)

    def read(self, bufs: td.GetBuffers, stream=None) -> ora.Batch:
        if stream is not None:
            stream.synchronize()
        else:
            torch.cuda.current_stream().synchronize()
        res = bufs.read_result()
        b = ora.Batch()
        b.n_samples, b.n_groups = res.n_samples, res.n_groups
        b.prompt_tokens, b.response_tokens, b.status = res.prompt_tokens, res.response_tokens, res.status
        k = b.n_samples
        b.indices = to_host(bufs.indices[:k])
        b.cu_prompt = to_host(bufs.cu_prompt[:k + 1])
        b.cu_response = to_host(bufs.cu_response[:k + 1])
        b.cu_seq = to_host(bufs.cu_seq[:k + 1])
        for c, t in bufs.cols.items():
            cls = self.dock.columns[c][1]
            if cls == td.SCALAR:
                b.columns[c] = to_host(t[:k])
            elif bufs.mode == td.PADDED:
                W = bufs.pad_prompt_to if cls == td.PROMPT else bufs.pad_response_to
                b.columns[c] = to_host(t[:k * W]).reshape(k, W)
            else:
                tot = b.prompt_tokens if cls == td.PROMPT else b.response_tokens
                b.columns[c] = to_host(t[:tot])
        if bufs.advantages is not None:
            b.advantages = to_host(bufs.advantages[:k])
        tot = int(b.prompt_tokens + b.response_tokens)
        if bufs.seq is not None:
            b.seq = to_host(bufs.seq[:tot])
        if bufs.seq_advantages is not None:
            b.seq_advantages = to_host(bufs.seq_advantages[:tot])
        return b

    # -- state ------------------------------------------------------------
    def table(self, which: int, index: int, dtype) -> np.ndarray:
        torch.cuda.synchronize()
        return self.dock.table(which, index).cpu().numpy().view(dtype).copy()


def assert_batch_equal(got: ora.Batch, want: ora.Batch, ctx=""):
    assert (got.n_samples, got.n_groups) == (want.n_samples, want.n_groups), ctx
    assert (got.prompt_tokens, got.response_tokens, got.status) == \
           (want.prompt_tokens, want.response_tokens, want.status), ctx
    assert np.array_equal(got.indices, want.indices), ctx
    assert np.array_equal(got.cu_prompt, want.cu_prompt), ctx
    assert np.array_equal(got.cu_response, want.cu_response), ctx
    assert np.array_equal(got.cu_seq, want.cu_seq), ctx
    assert sorted(got.columns) == sorted(want.columns), ctx
    for c in want.columns:
        assert H.bits_equal(got.columns[c], want.columns[c]), f"{ctx} column {c}"
    if want.advantages is None:
        assert got.advantages is None, ctx
    else:
        assert np.allclose(got.advantages.astype(np.float64), want.advantages.astype(np.float64),
                           rtol=REL_TOL, atol=ABS_TOL), ctx
        # a zero-variance group must come out as exact zeros on both sides
        assert np.array_equal(got.advantages == 0.0, want.advantages == 0.0), ctx
    assert (got.seq is None) == (want.seq is None) and (got.seq_advantages is None) == (want.seq_advantages is None), ctx
    if want.seq is not None:
        assert H.bits_equal(got.seq, want.seq), f"{ctx} fused stream"
    if want.seq_advantages is not None:
        assert np.allclose(got.seq_advantages.astype(np.float64), want.seq_advantages.astype(np.float64),
                           rtol=REL_TOL, atol=ABS_TOL), f"{ctx} stream advantages"
        # bit for bit the batch's own advantages over the response tokens, zero bits over the prompt
        lp = np.diff(got.cu_prompt).astype(np.int64)
        lr = np.diff(got.cu_response).astype(np.int64)
        mine = np.repeat(np.stack([np.zeros_like(got.advantages), got.advantages], axis=1).reshape(-1),
                         np.stack([lp, lr], axis=1).reshape(-1))
        assert H.bits_equal(got.seq_advantages, mine.astype(np.float32)), f"{ctx} stream advantages layout"


def _same(got: np.ndarray, want: np.ndarray, what: str):
    if not np.array_equal(got, want):
        bad = np.where(got != want)[0][:8]
        raise AssertionError(f"{what}: differs at {bad.tolist()}: got {got[bad].tolist()} want {want[bad].tolist()}")


def assert_state_equal(g: GpuDock, o: ora.OracleDock, arenas: bool = True, ctx=""):
    w = g.w
    rep = g.dock.validate()
    assert rep.violations == 0, f"{ctx} td_debug_validate: {rep.violations:#x} at {rep.first_sample}"
    _same(g.table(0, 0, np.uint32), o.status(), ctx + " status")
    for cls in (1, 2):
        _same(g.table(1, cls, np.int32), o.lengths(cls), ctx + f" len[{cls}]")
        _same(g.table(2, cls, np.int64), o.offsets(cls), ctx + f" off[{cls}]")
        _same(g.table(3, cls, np.uint64), o.cursors(cls), ctx + f" cursor[{cls}]")
    for c in range(len(w.consumers)):
        _same(g.table(4, c, np.uint32), o.claim_words(c), ctx + f" claim[{c}]")
        _same(g.table(5, c, np.uint32), o.consumed_words(c), ctx + f" consumed[{c}]")
    if arenas:
        for c, spec in enumerate(w.columns):
            dt = wl.DTYPE_NUMPY[spec.dtype]
            dev = g.table(6, c, dt)
            if spec.cls == wl.SCALAR:
                st = (o.status() >> c) & 1
                assert H.bits_equal(dev[st == 1], o.scalars(c)[st == 1]), ctx + f" scalars[{c}]"
                continue
            cls = H.CLS_NUM[spec.cls]
            cap = o.prompt_cap if cls == 1 else o.response_cap
            ln, off = o.lengths(cls), o.offsets(cls)
            stored = np.where((o.status() >> c) & 1)[0]
            for sh in range(w.S):
                a_dev = dev[sh * cap:(sh + 1) * cap]
                a_ora = o.arena(c, sh)
                # compare the bytes of stored rows (padding between rows is unspecified)
                mask = np.zeros(cap, dtype=bool)
                for s in stored:
                    if o.shard_of(int(s)) == sh:
                        mask[off[s]:off[s] + ln[s]] = True
                assert H.bits_equal(a_dev[mask], a_ora[mask]), ctx + f" arena[{c}][{sh}]"


def assert_stats_equal(g: GpuDock, o: ora.OracleDock, ctx=""):
    gs, os_ = g.dock.status(), o.stats()
    for f in ("n_oob", "n_dup", "n_len_mismatch", "n_arena_full", "n_truncated", "n_bad_length", "error_word"):
        assert getattr(gs, f) == getattr(os_, f), f"{ctx} {f}: {getattr(gs, f)} != {getattr(os_, f)}"
    for c in range(32):
        assert gs.put_accepted[c] == os_.put_accepted[c], f"{ctx} put_accepted[{c}]"
        assert gs.got_samples[c] == os_.got_samples[c], f"{ctx} got_samples[{c}]"
        assert gs.got_tokens[c] == os_.got_tokens[c], f"{ctx} got_tokens[{c}]"


def stream_args(w: wl.Workload, consumer: int) -> dict:
    """Keyword arguments that ask for the fused id stream (and, for a consumer with advantages,
    its advantage twin) on either side."""
    return dict(seq=(w.column_index("prompt_ids"), w.column_index("response_ids")),
                seq_adv=w.consumers[consumer].advantage)


def replay_both(w: wl.Workload, mode: int = td.PACKED, check_state_every: int = 0,
                max_get_checks: Optional[int] = None, arenas: bool = True, fused: bool = False):
    """Runs w.ops on the oracle and on the GPU in lock step, comparing every get; returns
    (gpu dock, oracle dock, batches)."""
    o = H.make_oracle(w)
    g = GpuDock(w)
    pad_p, pad_r = (w.pad_prompt_to, w.pad_response_to) if mode == td.PADDED else (0, 0)
    n_get = 0
    batches = []
    last = {}
    plans = {}
    pool_dev = {c: to_device(a, g.device) for c, a in w.pool.items()}
    for j, op in enumerate(w.ops):
        if op.kind == "put":
            cu, data = w.pack(op.column, op.indices)
            o.put(op.column, op.indices, cu, data)
            g.put(op.column, op.indices, cu, data)
        elif op.kind == "put_back":
            # the get of this consumer was enqueued just before; nothing has synchronised since
            want, bufs = last[op.consumer]
            g.dock.put_back(bufs, [(c, pool_dev[c]) for c in op.columns])
            H.oracle_put_back(w, o, want, op.columns)
            assert_batch_equal(g.read(bufs), want, f"op {j} consumer {op.consumer} (after write-back)")
        elif op.kind == "get_many":
            bufs = [g.buffers(c, op.max_samples, mode, pad_p, pad_r) for c in op.group]
            key = tuple(op.group)
            if key not in plans:
                plans[key] = g.dock.plan(bufs)
            g.dock.get_many(plans[key])                      # read back only after the write-backs are enqueued
            wants = [o.get(c, op.max_samples, mode, pad_p, pad_r) for c in op.group]
            for c, want, b in zip(op.group, wants, bufs):
                last[c] = (want, b)
                batches.append((c, want))
            nxt = w.ops[j + 1] if j + 1 < len(w.ops) else None
            if nxt is None or nxt.kind != "put_back_many":
                for c, want, b in zip(op.group, wants, bufs):
                    assert_batch_equal(g.read(b), want, f"op {j} consumer {c}")
        elif op.kind == "put_back_many":
            g.dock.put_back_many([(last[c][1], col, pool_dev[col]) for c, col in op.group])
            for c, col in op.group:
                H.oracle_put_back(w, o, last[c][0], [col])
            for c, (want, b) in last.items():
                assert_batch_equal(g.read(b), want, f"op {j} consumer {c} (after write-backs)")
        elif any(k.kind == "put_back" and k.consumer == op.consumer for k in w.ops[j + 1:j + 2]):
            want = o.get(op.consumer, op.max_samples, mode, pad_p, pad_r)
            bufs = g.buffers(op.consumer, op.max_samples, mode, pad_p, pad_r)
            g.dock.get(bufs)                         # not read back before the write-back is enqueued
            last[op.consumer] = (want, bufs)
            batches.append((op.consumer, want))
            n_get += 1
        else:
            if max_get_checks is not None and n_get >= max_get_checks:
                continue
            kw = stream_args(w, op.consumer) if fused else {}
            want = o.get(op.consumer, op.max_samples, mode, pad_p, pad_r, **kw)
            got = g.get(op.consumer, op.max_samples, mode, pad_p, pad_r, **kw)
            assert_batch_equal(got, want, f"op {j} consumer {op.consumer}")
            batches.append((op.consumer, want))
            n_get += 1
        if check_state_every and (j + 1) % check_state_every == 0:
            assert_state_equal(g, o, arenas=False, ctx=f"after op {j}")
    assert_state_equal(g, o, arenas=arenas, ctx="final")
    assert_stats_equal(g, o, "final")
    return g, o, batches
