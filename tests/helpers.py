"""Glue shared by the tests: build an oracle dock from a workload, replay a
schedule on it, and reference answers computed straight from the generator's
arrays (never from the oracle or the CUDA path)."""
from __future__ import annotations

from typing import Dict, List

import numpy as np

from oracle import td_oracle as ora
from paper_2507_19017_b200 import workloads as wl

CLS_NUM = {wl.SCALAR: 0, wl.PROMPT: 1, wl.RESPONSE: 2}


def make_oracle(w: wl.Workload, prompt_cap=None, response_cap=None, eps: float = 1e-6) -> ora.OracleDock:
    return ora.OracleDock(w.G, w.N, w.S, w.column_tuples(), w.consumer_tuples(),
                          prompt_cap if prompt_cap is not None else w.shard_capacity(wl.PROMPT),
                          response_cap if response_cap is not None else w.shard_capacity(wl.RESPONSE),
                          w.column_index("reward"), eps)


def back_rows(w: wl.Workload, column: int, batch) -> tuple:
    """What a worker state sends back for `batch`: (cu or None, data) cut from the workload's pool,
    row i of the batch at cu[i]."""
    k = batch.n_samples
    cls = w.columns[column].cls
    if cls == wl.SCALAR:
        return None, w.pool[column][:k]
    cu = batch.cu_prompt if cls == wl.PROMPT else batch.cu_response
    return np.ascontiguousarray(cu[:k + 1], dtype=np.int32), w.pool[column][:int(cu[k])]


def oracle_put_back(w: wl.Workload, dock: ora.OracleDock, batch, columns) -> None:
    """The oracle's statement of a write-back: an ordinary put of the batch's samples."""
    if batch.n_samples == 0:
        return
    for c in columns:
        cu, data = back_rows(w, c, batch)
        dock.put(c, batch.indices, cu, data)


def replay_oracle(w: wl.Workload, dock: ora.OracleDock, mode: int = ora.PACKED) -> List:
    """Run w.ops in order; returns the list of batches of the get ops."""
    out = []
    last = {}
    for op in w.ops:
        if op.kind == "put":
            cu, data = w.pack(op.column, op.indices)
            dock.put(op.column, op.indices, cu, data)
        elif op.kind == "put_back":
            oracle_put_back(w, dock, last[op.consumer], op.columns)
        elif op.kind == "get_many":            # one call: the consumers are served in order
            for c in op.group:
                out.append((c, dock.get(c, op.max_samples, mode, w.pad_prompt_to, w.pad_response_to)))
                last[c] = out[-1][1]
        elif op.kind == "put_back_many":       # one call: the write-backs are stored in order
            for c, col in op.group:
                oracle_put_back(w, dock, last[c], [col])
        else:
            out.append((op.consumer, dock.get(op.consumer, op.max_samples, mode,
                                              w.pad_prompt_to, w.pad_response_to)))
            last[op.consumer] = out[-1][1]
    return out


def expected_packed(w: wl.Workload, column: int, indices: np.ndarray) -> np.ndarray:
    """Rows of `indices` concatenated, taken from the generator's arrays."""
    spec = w.columns[column]
    src = w.data[spec.name]
    if spec.cls == wl.SCALAR:
        return src[np.asarray(indices, dtype=np.int64)]
    st = w.row_starts(spec.cls)
    parts = [src[st[s]:st[s + 1]] for s in indices]
    return np.concatenate(parts) if parts else np.zeros(0, src.dtype)


def expected_padded(w: wl.Workload, column: int, indices: np.ndarray, width: int, left: bool = False) -> np.ndarray:
    """The dense [len(indices), width] matrix of a ragged column from the generator's arrays: each
    row's elements at the row's start, or (left) flush with its end, the pad pattern elsewhere."""
    spec = w.columns[column]
    src = w.data[spec.name]
    st = w.row_starts(spec.cls)
    pad = np.array([spec.pad_bits], dtype=np.uint32).view(np.uint32)
    out = np.empty((len(indices), width), dtype=src.dtype)
    if src.dtype.itemsize == 4:
        out.view(np.uint32)[:] = np.uint32(spec.pad_bits)
    else:
        out.view(np.uint16)[:] = np.uint16(spec.pad_bits & 0xFFFF)
    for i, s in enumerate(indices):
        row = src[st[s]:st[s + 1]]
        if left:
            out[i, width - len(row):] = row
        else:
            out[i, :len(row)] = row
    del pad
    return out


def bits_equal(a: np.ndarray, b: np.ndarray) -> bool:
    """Raw-bit equality (payload is never interpreted: NaN and -0.0 must survive)."""
    a = np.ascontiguousarray(a)
    b = np.ascontiguousarray(b)
    if a.shape != b.shape or a.dtype.itemsize != b.dtype.itemsize:
        return False
    return a.view(np.uint8).tobytes() == b.view(np.uint8).tobytes()


def popcount_words(words: np.ndarray) -> int:
    return int(np.unpackbits(np.ascontiguousarray(words).view(np.uint8)).sum())


def bit_list(words: np.ndarray, count: int) -> np.ndarray:
    bits = np.unpackbits(np.ascontiguousarray(words).view(np.uint8), bitorder="little")
    return bits[:count].astype(bool)
