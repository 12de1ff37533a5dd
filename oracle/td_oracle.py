"""ctypes access to the CPU oracle (oracle/td_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg, never by the library.  This file marshals numpy
arrays into the C calls and holds no arithmetic of its own.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "td_oracle.c")
_LIB = os.path.join(_HERE, "libtd_oracle.so")

DTYPES = {"i32": 0, "f32": 1, "bf16": 2}
CLASSES = {"scalar": 0, "prompt": 1, "response": 2}
NP_DTYPE = {0: np.int32, 1: np.float32, 2: np.uint16}
PACKED, PADDED = 0, 1
OUT_LEFT_PAD_PROMPT = 1            # flag of a get's output: prompt rows end at their width (PADDED only)
F_ADVANTAGE = 1

ERR_OOB_INDEX, ERR_DUP_PUT, ERR_LEN_MISMATCH, ERR_ARENA_FULL, ERR_OUT_TRUNC = 1, 2, 4, 8, 16
ERR_BAD_LENGTH = 64


_LIB_SAN = os.path.join(_HERE, "libtd_oracle_san.so")
SANITIZED_ENV = "TD_ORACLE_SANITIZED"      # set: lib() loads the build below instead of the plain one


def build(force: bool = False, sanitize: bool = False) -> str:
    """Compile the oracle with gcc (no optimisation flags beyond -O2).  sanitize: a second build
    with AddressSanitizer and UndefinedBehaviorSanitizer (errors abort), for the test that runs
    the oracle's own pins under them; the process that loads it must have libasan preloaded."""
    hdr = os.path.join(_HERE, "td_oracle.h")
    out = _LIB_SAN if sanitize else _LIB
    stale = (not os.path.exists(out)
             or os.path.getmtime(out) < max(os.path.getmtime(_SRC), os.path.getmtime(hdr)))
    if force or stale:
        extra = (["-g", "-O1", "-fno-omit-frame-pointer", "-fsanitize=address,undefined",
                  "-fno-sanitize-recover=all"] if sanitize else ["-O2"])
        subprocess.check_call(["gcc", *extra, "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC",
                               "-o", out, _SRC, "-lm"])
    return out


class _Column(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("cls", C.c_int32), ("pad_bits", C.c_uint32)]


class _Consumer(C.Structure):
    _fields_ = [("need_mask", C.c_uint32), ("out_mask", C.c_uint32), ("flags", C.c_uint32)]


class _Config(C.Structure):
    _fields_ = [("n_prompts", C.c_uint32), ("n_per_group", C.c_uint32), ("n_shards", C.c_uint32),
                ("n_columns", C.c_uint32), ("columns", C.POINTER(_Column)),
                ("n_consumers", C.c_uint32), ("consumers", C.POINTER(_Consumer)),
                ("prompt_elems_per_shard", C.c_uint64), ("response_elems_per_shard", C.c_uint64),
                ("reward_column", C.c_uint32), ("adv_eps", C.c_float)]


class _Result(C.Structure):
    _fields_ = [("n_samples", C.c_uint32), ("n_groups", C.c_uint32),
                ("prompt_tokens", C.c_uint64), ("response_tokens", C.c_uint64),
                ("status", C.c_uint32)]


class _GetOut(C.Structure):
    _fields_ = [("mode", C.c_int32), ("pad_prompt_to", C.c_uint32), ("pad_response_to", C.c_uint32),
                ("flags", C.c_uint32), ("indices", C.c_void_p), ("cu_prompt", C.c_void_p), ("cu_response", C.c_void_p),
                ("cu_seq", C.c_void_p), ("col", C.c_void_p * 32),
                ("col_capacity_elems", C.c_uint64 * 32), ("advantages", C.c_void_p),
                ("result", C.POINTER(_Result)),
                ("seq_prompt_col", C.c_uint32), ("seq_response_col", C.c_uint32), ("seq", C.c_void_p),
                ("seq_capacity_elems", C.c_uint64), ("seq_advantages", C.c_void_p)]


class _Stats(C.Structure):
    _fields_ = [("put_accepted", C.c_uint64 * 32), ("got_samples", C.c_uint64 * 32),
                ("got_tokens", C.c_uint64 * 32), ("n_oob", C.c_uint64), ("n_dup", C.c_uint64),
                ("n_len_mismatch", C.c_uint64), ("n_arena_full", C.c_uint64),
                ("n_truncated", C.c_uint64), ("n_bad_length", C.c_uint64),
                ("error_word", C.c_uint32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build(sanitize=bool(os.environ.get(SANITIZED_ENV))))
        L.ora_create.restype = C.c_void_p
        L.ora_create.argtypes = [C.POINTER(_Config)]
        L.ora_destroy.argtypes = [C.c_void_p]
        L.ora_reset.argtypes = [C.c_void_p]
        L.ora_put.restype = C.c_int64
        L.ora_put.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p]
        L.ora_get.restype = C.c_int
        L.ora_get.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.POINTER(_GetOut)]
        L.ora_gather.restype = C.c_int
        L.ora_gather.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.POINTER(_GetOut)]
        L.ora_get_stats.argtypes = [C.c_void_p, C.POINTER(_Stats)]
        L.ora_shard_of.restype = C.c_uint32
        L.ora_shard_of.argtypes = [C.c_void_p, C.c_uint32]
        for nm in ("ora_status", "ora_len", "ora_off", "ora_cursor", "ora_claim", "ora_consumed",
                   "ora_arena", "ora_scalars"):
            getattr(L, nm).restype = C.c_void_p
        L.ora_status.argtypes = [C.c_void_p]
        L.ora_len.argtypes = [C.c_void_p, C.c_int]
        L.ora_off.argtypes = [C.c_void_p, C.c_int]
        L.ora_cursor.argtypes = [C.c_void_p, C.c_int]
        L.ora_claim.argtypes = [C.c_void_p, C.c_uint32]
        L.ora_consumed.argtypes = [C.c_void_p, C.c_uint32]
        L.ora_arena.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32]
        L.ora_scalars.argtypes = [C.c_void_p, C.c_uint32]
        for nm in ("ora_cv", "ora_tcv"):
            getattr(L, nm).restype = C.c_double
            getattr(L, nm).argtypes = [C.c_double] * 7
        L.ora_tcv_dock.restype = C.c_double
        L.ora_tcv_dock.argtypes = [C.c_double] * 9
        _lib = L
    return _lib


def _view(ptr: int, dtype, count: int) -> np.ndarray:
    if count == 0 or not ptr:
        return np.zeros(0, dtype=dtype)
    buf = (C.c_uint8 * (count * np.dtype(dtype).itemsize)).from_address(ptr)
    return np.frombuffer(buf, dtype=dtype, count=count).copy()


class Batch:
    """What one get returned: numpy copies trimmed to the valid sizes."""

    def __init__(self):
        self.n_samples = 0
        self.n_groups = 0
        self.prompt_tokens = 0
        self.response_tokens = 0
        self.status = 0
        self.indices: np.ndarray = np.zeros(0, np.int32)
        self.cu_prompt: np.ndarray = np.zeros(1, np.int32)
        self.cu_response: np.ndarray = np.zeros(1, np.int32)
        self.cu_seq: np.ndarray = np.zeros(1, np.int32)
        self.columns: Dict[int, np.ndarray] = {}
        self.advantages: Optional[np.ndarray] = None
        self.seq: Optional[np.ndarray] = None              # fused prompt+response stream, by cu_seq
        self.seq_advantages: Optional[np.ndarray] = None   # same layout: 0 on prompt tokens, A on response tokens


class OracleDock:
    """columns: sequence of (dtype_tag, class_tag, pad_bits); consumers: sequence of
    (need_mask, out_mask, advantage_flag)."""

    def __init__(self, G: int, N: int, S: int, columns: Sequence, consumers: Sequence,
                 prompt_cap: int, response_cap: int, reward_column: int, eps: float = 1e-6):
        self.G, self.N, self.S, self.n = G, N, S, G * N
        self.columns = [(DTYPES[d], CLASSES[c], int(p)) for d, c, p in columns]
        self.consumers = [(int(a), int(b), F_ADVANTAGE if f else 0) for a, b, f in consumers]
        cols = (_Column * len(self.columns))(*[_Column(*c) for c in self.columns])
        cons = (_Consumer * len(self.consumers))(*[_Consumer(*c) for c in self.consumers])
        cfg = _Config(G, N, S, len(self.columns), cols, len(self.consumers), cons,
                      prompt_cap, response_cap, reward_column, eps)
        self._h = lib().ora_create(C.byref(cfg))
        if not self._h:
            raise ValueError("ora_create rejected the configuration")
        self.prompt_cap = (prompt_cap + 7) // 8 * 8
        self.response_cap = (response_cap + 7) // 8 * 8

    def close(self):
        if self._h:
            lib().ora_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        lib().ora_reset(self._h)

    def put(self, column: int, indices: np.ndarray, cu: Optional[np.ndarray], data: np.ndarray) -> int:
        idx = np.ascontiguousarray(indices, dtype=np.int32)
        dat = np.ascontiguousarray(data)
        cup = None
        if cu is not None:
            cua = np.ascontiguousarray(cu, dtype=np.int32)
            cup = cua.ctypes.data
        return lib().ora_put(self._h, column, idx.ctypes.data, len(idx), cup, dat.ctypes.data)

    # -- get / gather -----------------------------------------------------
    def _alloc(self, consumer: int, max_samples: int, mode: int, pad_p: int, pad_r: int,
               capacities: Optional[Dict[int, int]], want: Optional[Sequence[int]],
               lens_bound: Sequence[int], seq=None, seq_adv: bool = False, seq_cap: Optional[int] = None,
               out_flags: int = 0):
        need, outm, flags = self.consumers[consumer]
        res = _Result()
        go = _GetOut()
        go.mode, go.pad_prompt_to, go.pad_response_to, go.flags = mode, pad_p, pad_r, out_flags
        bufs = {"indices": np.zeros(max_samples, np.int32)}
        for nm in ("cu_prompt", "cu_response", "cu_seq"):
            bufs[nm] = np.zeros(max_samples + 1, np.int32)
        go.indices = bufs["indices"].ctypes.data
        go.cu_prompt = bufs["cu_prompt"].ctypes.data
        go.cu_response = bufs["cu_response"].ctypes.data
        go.cu_seq = bufs["cu_seq"].ctypes.data
        cols = {}
        for c, (dt, cls, _pad) in enumerate(self.columns):
            if not (outm >> c) & 1:
                continue
            if want is not None and c not in want:
                continue
            if capacities is not None and c in capacities:
                cap = int(capacities[c])
            elif cls == 0:
                cap = max_samples
            elif mode == PADDED:
                cap = max_samples * (pad_p if cls == 1 else pad_r)
            else:
                cap = int(lens_bound[cls])
            cols[c] = np.zeros(max(cap, 1), NP_DTYPE[dt])
            go.col[c] = cols[c].ctypes.data
            go.col_capacity_elems[c] = cap
        adv = None
        if flags & F_ADVANTAGE:
            adv = np.zeros(max_samples, np.float32)
            go.advantages = adv.ctypes.data
        go.result = C.pointer(res)
        if seq is not None or seq_adv:
            cap = int(seq_cap) if seq_cap is not None else int(lens_bound[1]) + int(lens_bound[2])
            go.seq_capacity_elems = cap
            if seq is not None:
                go.seq_prompt_col, go.seq_response_col = seq
                bufs["seq"] = np.zeros(max(cap, 1), NP_DTYPE[self.columns[seq[0]][0]])
                go.seq = bufs["seq"].ctypes.data
            if seq_adv:
                bufs["seq_advantages"] = np.zeros(max(cap, 1), np.float32)
                go.seq_advantages = bufs["seq_advantages"].ctypes.data
        return go, res, bufs, cols, adv

    def _finish(self, go, res, bufs, cols, adv, mode, pad_p, pad_r) -> Batch:
        b = Batch()
        b.n_samples, b.n_groups = res.n_samples, res.n_groups
        b.prompt_tokens, b.response_tokens, b.status = res.prompt_tokens, res.response_tokens, res.status
        k = b.n_samples
        b.indices = bufs["indices"][:k].copy()
        b.cu_prompt = bufs["cu_prompt"][:k + 1].copy()
        b.cu_response = bufs["cu_response"][:k + 1].copy()
        b.cu_seq = bufs["cu_seq"][:k + 1].copy()
        for c, a in cols.items():
            cls = self.columns[c][1]
            if cls == 0:
                b.columns[c] = a[:k].copy()
            elif mode == PADDED:
                W = pad_p if cls == 1 else pad_r
                b.columns[c] = a[:k * W].reshape(k, W).copy()
            else:
                tot = b.prompt_tokens if cls == 1 else b.response_tokens
                b.columns[c] = a[:tot].copy()
        if adv is not None:
            b.advantages = adv[:k].copy()
        tot = int(b.prompt_tokens + b.response_tokens)
        if "seq" in bufs:
            b.seq = bufs["seq"][:tot].copy()
        if "seq_advantages" in bufs:
            b.seq_advantages = bufs["seq_advantages"][:tot].copy()
        return b

    def _bounds(self, max_samples: int) -> List[int]:
        """Upper bounds on packed tokens for max_samples samples, by length class."""
        out = [0, 0, 0]
        for cls in (1, 2):
            ln = self.lengths(cls)
            pos = np.sort(np.maximum(ln, 0))[::-1]
            out[cls] = int(pos[:max_samples].sum(dtype=np.int64))
        return out

    def get(self, consumer: int, max_samples: int, mode: int = PACKED, pad_prompt_to: int = 0,
            pad_response_to: int = 0, capacities: Optional[Dict[int, int]] = None,
            want: Optional[Sequence[int]] = None, seq=None, seq_adv: bool = False,
            seq_cap: Optional[int] = None, out_flags: int = 0) -> Batch:
        """seq = (prompt column, response column) asks for the fused token stream, seq_adv for
        its advantage twin; seq_cap bounds both (default: room for the longest rows).
        out_flags = OUT_LEFT_PAD_PROMPT: padded prompt rows carry their pad in front."""
        ragged = [c for c, (_d, cls, _p) in enumerate(self.columns)
                  if cls != 0 and (self.consumers[consumer][1] >> c) & 1 and (want is None or c in want)]
        need_bound = mode == PACKED and any(capacities is None or c not in capacities for c in ragged)
        need_bound = need_bound or ((seq is not None or seq_adv) and seq_cap is None)
        bound = self._bounds(max_samples) if need_bound else [0, 0, 0]
        go, res, bufs, cols, adv = self._alloc(consumer, max_samples, mode, pad_prompt_to,
                                               pad_response_to, capacities, want, bound, seq, seq_adv, seq_cap,
                                               out_flags)
        rc = lib().ora_get(self._h, consumer, max_samples, C.byref(go))
        if rc != 0:
            raise ValueError("ora_get: bad argument")
        return self._finish(go, res, bufs, cols, adv, mode, pad_prompt_to, pad_response_to)

    def prepare_get(self, consumer: int, max_samples: int, capacities: Dict[int, int], mode: int = PACKED,
                    pad_prompt_to: int = 0, pad_response_to: int = 0):
        """Output buffers allocated once, for callers that time ora_get itself."""
        return self._alloc(consumer, max_samples, mode, pad_prompt_to, pad_response_to, capacities,
                           None, [0, 0, 0]) + (consumer, max_samples)

    def get_prepared(self, prepared) -> int:
        """ora_get into buffers from prepare_get(); returns the number of samples served."""
        go, res = prepared[0], prepared[1]
        if lib().ora_get(self._h, prepared[5], prepared[6], C.byref(go)) != 0:
            raise ValueError("ora_get: bad argument")
        return res.n_samples

    def put_raw(self, column: int, idx: np.ndarray, cu: Optional[np.ndarray], data: np.ndarray) -> int:
        """ora_put on arrays that already have the right dtype and layout (no conversion)."""
        return lib().ora_put(self._h, column, idx.ctypes.data, len(idx),
                             cu.ctypes.data if cu is not None else None, data.ctypes.data)

    def gather(self, consumer: int, indices: np.ndarray, mode: int = PACKED, pad_prompt_to: int = 0,
               pad_response_to: int = 0, want: Optional[Sequence[int]] = None, seq=None,
               seq_adv: bool = False, out_flags: int = 0) -> Batch:
        idx = np.ascontiguousarray(indices, dtype=np.int32)
        k = len(idx)
        bound = [0, 0, 0]
        for cls in (1, 2):
            bound[cls] = int(np.maximum(self.lengths(cls)[idx], 0).sum(dtype=np.int64)) if k else 0
        go, res, bufs, cols, adv = self._alloc(consumer, max(k, 1), mode, pad_prompt_to,
                                               pad_response_to, None, want, bound, seq, seq_adv, None, out_flags)
        rc = lib().ora_gather(self._h, consumer, idx.ctypes.data, k, C.byref(go))
        if rc != 0:
            raise ValueError("ora_gather: bad argument")
        return self._finish(go, res, bufs, cols, adv, mode, pad_prompt_to, pad_response_to)

    # -- state ------------------------------------------------------------
    def stats(self) -> _Stats:
        st = _Stats()
        lib().ora_get_stats(self._h, C.byref(st))
        return st

    def shard_of(self, s: int) -> int:
        return lib().ora_shard_of(self._h, s)

    def status(self) -> np.ndarray:
        return _view(lib().ora_status(self._h), np.uint32, self.n)

    def lengths(self, cls: int) -> np.ndarray:
        return _view(lib().ora_len(self._h, cls), np.int32, self.n)

    def offsets(self, cls: int) -> np.ndarray:
        return _view(lib().ora_off(self._h, cls), np.int64, self.n)

    def cursors(self, cls: int) -> np.ndarray:
        return _view(lib().ora_cursor(self._h, cls), np.uint64, self.S)

    def claim_words(self, consumer: int) -> np.ndarray:
        return _view(lib().ora_claim(self._h, consumer), np.uint32, (self.G + 31) // 32)

    def consumed_words(self, consumer: int) -> np.ndarray:
        return _view(lib().ora_consumed(self._h, consumer), np.uint32, (self.n + 31) // 32)

    def arena(self, column: int, shard: int) -> np.ndarray:
        dt, cls, _ = self.columns[column]
        cap = self.prompt_cap if cls == 1 else self.response_cap
        return _view(lib().ora_arena(self._h, column, shard), NP_DTYPE[dt], cap)

    def scalars(self, column: int) -> np.ndarray:
        dt, _, _ = self.columns[column]
        return _view(lib().ora_scalars(self._h, column), NP_DTYPE[dt], self.n)


def cv(G, N, B, PL, n, SL, M) -> float:
    return lib().ora_cv(G, N, B, PL, n, SL, M)


def tcv(G, N, B, PL, n, SL, M) -> float:
    return lib().ora_tcv(G, N, B, PL, n, SL, M)


def tcv_dock(G, N, B, PL, n, SL, M, Cn, S) -> float:
    return lib().ora_tcv_dock(G, N, B, PL, n, SL, M, Cn, S)
