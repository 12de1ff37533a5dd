"""Thin ctypes binding of the C ABI in include/td.h.

Argument marshalling only: every step of put and get runs in the CUDA library.  PyTorch
supplies device memory (`torch.empty(...).data_ptr()`) and streams; nothing here computes
on tensors.  There is no CPU fallback: if libtd.so cannot be loaded, or a call fails,
an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence, Tuple

from . import build as _build

I32, F32, BF16 = 0, 1, 2
SCALAR, PROMPT, RESPONSE = 0, 1, 2
PACKED, PADDED = 0, 1
OUT_LEFT_PAD_PROMPT = 1            # td_get_out.flags
F_ADVANTAGE = 1
OK, EINVAL, EWORKSPACE, ECUDA, ETOOLARGE = 0, -1, -2, -3, -4
ERR_OOB_INDEX, ERR_DUP_PUT, ERR_LEN_MISMATCH, ERR_ARENA_FULL = 1, 2, 4, 8
ERR_OUT_TRUNCATED, ERR_LOOKBACK_TIMEOUT, ERR_BAD_LENGTH, ERR_COPY_TIMEOUT = 16, 32, 64, 128
(BAD_STORED_WITHOUT_ROW, BAD_ROW_PLACEMENT, BAD_ROW_OVERLAP, BAD_STATUS_BITS, BAD_SERVED_UNCLAIMED,
 BAD_SERVED_NOT_READY, BAD_COUNTERS) = 1, 2, 4, 8, 16, 32, 64          # td_debug_validate

DTYPE_TAG = {"i32": I32, "f32": F32, "bf16": BF16}
CLASS_TAG = {"scalar": SCALAR, "prompt": PROMPT, "response": RESPONSE}
ELEM_SIZE = {I32: 4, F32: 4, BF16: 2}

# every symbol include/td.h declares
EXPORTS = ["td_query_workspace", "td_create", "td_destroy", "td_put", "td_get",
           "td_get_scratch_bytes", "td_reset", "td_status", "td_debug_table",
           "td_launch_count", "td_strerror", "td_kernel_timing", "td_kernel_timing_read",
           "td_put_host_stage_bytes", "td_put_host", "td_get_host", "td_put_many",
           "td_plan_bytes", "td_plan_create", "td_plan_destroy", "td_get_many", "td_get_static",
           "td_model_bytes", "td_put_back", "td_put_back_many", "td_put_many_host", "td_get_many_host", "td_get_many_host_stage_bytes", "td_debug_validate",
           "td_debug_lookback"]


class TdModel(C.Structure):
    _fields_ = [(k, C.c_uint64) for k in ("G", "N", "PL", "n", "SL", "M", "B", "C", "S")]


class TdColumn(C.Structure):
    _fields_ = [("name", C.c_char_p), ("dtype", C.c_int32), ("cls", C.c_int32), ("pad_bits", C.c_uint32)]


class TdConsumer(C.Structure):
    _fields_ = [("name", C.c_char_p), ("need_mask", C.c_uint32), ("out_mask", C.c_uint32),
                ("flags", C.c_uint32)]


class TdConfig(C.Structure):
    _fields_ = [("n_prompts", C.c_uint32), ("n_per_group", C.c_uint32), ("n_shards", C.c_uint32),
                ("n_columns", C.c_uint32), ("columns", C.POINTER(TdColumn)),
                ("n_consumers", C.c_uint32), ("consumers", C.POINTER(TdConsumer)),
                ("prompt_elems_per_shard", C.c_uint64), ("response_elems_per_shard", C.c_uint64),
                ("reward_column", C.c_uint32), ("adv_eps", C.c_float), ("device", C.c_int32)]


class TdResult(C.Structure):
    _fields_ = [("n_samples", C.c_uint32), ("n_groups", C.c_uint32),
                ("prompt_tokens", C.c_uint64), ("response_tokens", C.c_uint64),
                ("status", C.c_uint32), ("reserved", C.c_uint32)]


class TdGetOut(C.Structure):
    _fields_ = [("mode", C.c_int32), ("pad_prompt_to", C.c_uint32), ("pad_response_to", C.c_uint32),
                ("flags", C.c_uint32),
                ("indices", C.c_void_p), ("cu_prompt", C.c_void_p), ("cu_response", C.c_void_p),
                ("cu_seq", C.c_void_p), ("col", C.c_void_p * 32),
                ("col_capacity_elems", C.c_uint64 * 32), ("advantages", C.c_void_p),
                ("result", C.c_void_p), ("scratch", C.c_void_p), ("scratch_bytes", C.c_uint64),
                ("seq_prompt_col", C.c_uint32), ("seq_response_col", C.c_uint32), ("seq", C.c_void_p),
                ("seq_capacity_elems", C.c_uint64), ("seq_advantages", C.c_void_p)]


class TdPutItem(C.Structure):
    _fields_ = [("column", C.c_uint32), ("k", C.c_uint32), ("d_indices", C.c_void_p),
                ("d_cu", C.c_void_p), ("d_data", C.c_void_p), ("data_elems", C.c_uint64)]


class TdBackItem(C.Structure):
    _fields_ = [("column", C.c_uint32), ("reserved", C.c_uint32), ("d_data", C.c_void_p),
                ("data_elems", C.c_uint64)]


class TdBackReq(C.Structure):
    _fields_ = [("batch", C.c_void_p), ("max_samples", C.c_uint32), ("column", C.c_uint32),
                ("d_data", C.c_void_p), ("data_elems", C.c_uint64)]


class TdValidateReport(C.Structure):
    _fields_ = [("violations", C.c_uint32), ("reserved", C.c_uint32), ("first_sample", C.c_uint64),
                ("stored", C.c_uint64 * 32), ("served", C.c_uint64 * 32), ("arena_elems_used", C.c_uint64 * 3)]


class TdGetReq(C.Structure):
    _fields_ = [("consumer", C.c_uint32), ("max_samples", C.c_uint32), ("out", TdGetOut)]


class TdStats(C.Structure):
    _fields_ = [("put_accepted", C.c_uint64 * 32), ("got_samples", C.c_uint64 * 32),
                ("got_tokens", C.c_uint64 * 32), ("n_oob", C.c_uint64), ("n_dup", C.c_uint64),
                ("n_len_mismatch", C.c_uint64), ("n_arena_full", C.c_uint64),
                ("n_truncated", C.c_uint64), ("n_bad_length", C.c_uint64),
                ("n_claim_conflicts", C.c_uint64), ("n_lookback_timeouts", C.c_uint64),
                ("error_word", C.c_uint32), ("reserved", C.c_uint32)]


class TdError(RuntimeError):
    def __init__(self, call: str, code: int):
        self.code = code
        msg = lib().td_strerror(code).decode() if _lib is not None else "?"
        super().__init__(f"{call} failed: {code} ({msg})")


_lib = None


def lib_path() -> str:
    """The library to load: libtd.so beside this file, or the build named by TD_LIB_PATH (a build
    of the same sources with other compiler flags: sanitizers, NVTX ranges)."""
    return os.environ.get("TD_LIB_PATH") or _build.LIB_PATH


def lib():
    """Loads libtd.so (raises if it is missing: there is no other implementation)."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with "
                               "`python -m paper_2507_19017_b200.build` (needs nvcc)")
        L = C.CDLL(path)
        vp, u32, u64 = C.c_void_p, C.c_uint32, C.c_uint64
        L.td_query_workspace.restype = C.c_int
        L.td_query_workspace.argtypes = [C.POINTER(TdConfig), C.POINTER(C.c_size_t)]
        L.td_create.restype = C.c_int
        L.td_create.argtypes = [C.POINTER(TdConfig), vp, C.c_size_t, C.POINTER(vp)]
        L.td_destroy.restype = C.c_int
        L.td_destroy.argtypes = [vp]
        L.td_put.restype = C.c_int
        L.td_put.argtypes = [vp, u32, vp, u32, vp, vp, u64, vp]
        L.td_get.restype = C.c_int
        L.td_get.argtypes = [vp, u32, u32, C.POINTER(TdGetOut), vp]
        L.td_get_scratch_bytes.restype = C.c_size_t
        L.td_get_scratch_bytes.argtypes = [vp]
        L.td_reset.restype = C.c_int
        L.td_reset.argtypes = [vp, vp]
        L.td_status.restype = C.c_int
        L.td_status.argtypes = [vp, C.POINTER(TdStats), vp]
        L.td_debug_table.restype = C.c_int
        L.td_debug_table.argtypes = [vp, C.c_int, u32, C.POINTER(vp), C.POINTER(C.c_size_t)]
        L.td_launch_count.restype = u64
        L.td_launch_count.argtypes = [vp]
        L.td_strerror.restype = C.c_char_p
        L.td_strerror.argtypes = [C.c_int]
        L.td_kernel_timing.restype = C.c_int
        L.td_kernel_timing.argtypes = [vp, C.c_int]
        L.td_kernel_timing_read.restype = C.c_int
        L.td_kernel_timing_read.argtypes = [vp, C.c_int, C.POINTER(u64), C.POINTER(C.c_double)]
        L.td_put_host_stage_bytes.restype = C.c_size_t
        L.td_put_host_stage_bytes.argtypes = [vp, u32, u32, u64]
        L.td_put_host.restype = C.c_int
        L.td_put_host.argtypes = [vp, u32, vp, u32, vp, vp, u64, vp, C.c_size_t, vp]
        L.td_get_host.restype = C.c_int
        L.td_get_host.argtypes = [vp, u32, u32, C.POINTER(TdGetOut), C.POINTER(TdGetOut), vp]
        L.td_put_many.restype = C.c_int
        L.td_put_many.argtypes = [vp, C.POINTER(TdPutItem), u32, vp]
        L.td_put_back.restype = C.c_int
        L.td_put_back.argtypes = [vp, C.POINTER(TdGetOut), u32, C.POINTER(TdBackItem), u32, vp]
        L.td_put_back_many.restype = C.c_int
        L.td_put_back_many.argtypes = [vp, C.POINTER(TdBackReq), u32, vp]
        L.td_put_many_host.restype = C.c_int
        L.td_put_many_host.argtypes = [vp, C.POINTER(TdPutItem), u32, vp, C.c_size_t, vp]
        L.td_get_many_host.restype = C.c_int
        L.td_get_many_host.argtypes = [vp, vp, C.POINTER(TdGetOut), u32, vp, C.c_size_t, vp]
        L.td_get_many_host_stage_bytes.restype = C.c_size_t
        L.td_get_many_host_stage_bytes.argtypes = [vp]
        L.td_debug_validate.restype = C.c_int
        L.td_debug_validate.argtypes = [vp, vp, C.POINTER(TdValidateReport)]
        L.td_debug_lookback.restype = C.c_int
        L.td_debug_lookback.argtypes = [vp, u32, u32]
        L.td_plan_bytes.restype = C.c_size_t
        L.td_plan_bytes.argtypes = [vp, u32]
        L.td_plan_create.restype = C.c_int
        L.td_plan_create.argtypes = [vp, C.POINTER(TdGetReq), u32, vp, C.c_size_t, vp, C.POINTER(vp)]
        L.td_plan_destroy.restype = C.c_int
        L.td_plan_destroy.argtypes = [vp]
        L.td_get_many.restype = C.c_int
        L.td_get_many.argtypes = [vp, vp, vp]
        L.td_get_static.restype = C.c_int
        L.td_get_static.argtypes = [vp, u32, u32, C.POINTER(TdGetOut), vp]
        L.td_model_bytes.restype = C.c_int
        L.td_model_bytes.argtypes = [C.POINTER(TdModel), C.POINTER(u64), C.POINTER(u64), C.POINTER(C.c_double)]
        _lib = L
    return _lib


def model_bytes(G, N, PL, n, SL, M, B=4, C_=0, S=1):
    """Eq. 1, Eq. 2 and Eq. 4 of the paper's volume model, in bytes: (cv, tcv, tcv_dock)."""
    m = TdModel(G, N, PL, n, SL, M, B, C_, S)
    cv, tcv, dock = C.c_uint64(), C.c_uint64(), C.c_double()
    _check("td_model_bytes", lib().td_model_bytes(C.byref(m), C.byref(cv), C.byref(tcv), C.byref(dock)))
    return cv.value, tcv.value, dock.value


def _check(call: str, rc: int):
    if rc != 0:
        raise TdError(call, rc)


def make_config(G: int, N: int, S: int, columns: Sequence[Tuple[str, str, int]],
                consumers: Sequence[Tuple[int, int, bool]], prompt_cap: int, response_cap: int,
                reward_column: int, eps: float = 1e-6, device: int = 0):
    """columns: (dtype tag, class tag, pad_bits); consumers: (need_mask, out_mask, advantage).
    Returns (TdConfig, keepalive) - keep the second value alive as long as the first."""
    cols = (TdColumn * len(columns))(*[TdColumn(None, DTYPE_TAG[d], CLASS_TAG[c], int(p))
                                       for d, c, p in columns])
    cons = (TdConsumer * len(consumers))(*[TdConsumer(None, int(a), int(b), F_ADVANTAGE if f else 0)
                                           for a, b, f in consumers])
    cfg = TdConfig(G, N, S, len(columns), cols, len(consumers), cons, prompt_cap, response_cap,
                   reward_column, eps, device)
    return cfg, (cols, cons)


def query_workspace(cfg: TdConfig) -> int:
    out = C.c_size_t(0)
    _check("td_query_workspace", lib().td_query_workspace(C.byref(cfg), C.byref(out)))
    return out.value


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class GetBuffers:
    """Device buffers of one get, allocated once and reusable for any number of calls."""

    def __init__(self, dock: "Dock", consumer: int, max_samples: int, mode: int = PACKED,
                 pad_prompt_to: int = 0, pad_response_to: int = 0,
                 capacities: Optional[Dict[int, int]] = None, want: Optional[Sequence[int]] = None,
                 prompt_tokens_cap: Optional[int] = None, response_tokens_cap: Optional[int] = None,
                 seq: Optional[Tuple[int, int]] = None, seq_adv: bool = False, seq_cap: Optional[int] = None,
                 host_payload: bool = False, left_pad_prompts: bool = False):
        """seq = (prompt column, response column) adds the fused token stream, seq_adv its
        advantage twin; seq_cap is the room behind each (default: both token caps together).
        left_pad_prompts (PADDED mode): prompt rows end at their width, the pad in front.
        host_payload: the column buffers (and the stream) are pinned host memory that the device
        writes directly; indices, cu_seqlens, advantages and the result block stay on the device."""
        import torch
        dev = dock.device
        self.host_payload = host_payload

        def payload(n, dtype):
            if host_payload:
                return torch.empty(n, dtype=dtype, pin_memory=True)
            return torch.empty(n, dtype=dtype, device=dev)

        self.dock, self.consumer, self.max_samples, self.mode = dock, consumer, max_samples, mode
        self.pad_prompt_to, self.pad_response_to = pad_prompt_to, pad_response_to
        self.flags = OUT_LEFT_PAD_PROMPT if left_pad_prompts else 0
        i32 = torch.int32
        self.indices = torch.zeros(max_samples, dtype=i32, device=dev)
        self.cu_prompt = torch.zeros(max_samples + 1, dtype=i32, device=dev)
        self.cu_response = torch.zeros(max_samples + 1, dtype=i32, device=dev)
        self.cu_seq = torch.zeros(max_samples + 1, dtype=i32, device=dev)
        self.result = torch.zeros(C.sizeof(TdResult), dtype=torch.uint8, device=dev)
        self.scratch = torch.zeros(lib().td_get_scratch_bytes(dock.handle), dtype=torch.uint8, device=dev)
        need, outm, adv = dock.consumers[consumer]
        self.advantages = torch.zeros(max_samples, dtype=torch.float32, device=dev) if adv else None
        self.cols: Dict[int, "torch.Tensor"] = {}
        self.caps: Dict[int, int] = {}
        tdt = {I32: torch.int32, F32: torch.float32, BF16: torch.bfloat16}
        for c, (dt, cls, _pad) in enumerate(dock.columns):
            if not (outm >> c) & 1 or (want is not None and c not in want):
                continue
            if capacities is not None and c in capacities:
                cap = int(capacities[c])
            elif cls == SCALAR:
                cap = max_samples
            elif mode == PADDED:
                cap = max_samples * (pad_prompt_to if cls == PROMPT else pad_response_to)
            else:
                cap = prompt_tokens_cap if cls == PROMPT else response_tokens_cap
                if cap is None:
                    raise ValueError("packed ragged columns need prompt_tokens_cap / response_tokens_cap "
                                     "or explicit capacities")
            self.caps[c] = cap
            self.cols[c] = payload(max(cap, 1), tdt[dt])
        go = TdGetOut()
        go.mode, go.pad_prompt_to, go.pad_response_to = mode, pad_prompt_to, pad_response_to
        go.flags = self.flags
        go.indices, go.cu_prompt = self.indices.data_ptr(), self.cu_prompt.data_ptr()
        go.cu_response, go.cu_seq = self.cu_response.data_ptr(), self.cu_seq.data_ptr()
        for c, t in self.cols.items():
            go.col[c] = t.data_ptr()
            go.col_capacity_elems[c] = self.caps[c]
        go.advantages = self.advantages.data_ptr() if self.advantages is not None else None
        go.result = self.result.data_ptr()
        go.scratch, go.scratch_bytes = self.scratch.data_ptr(), self.scratch.numel()
        self.seq = self.seq_advantages = None
        if seq is not None or seq_adv:
            cap = int(seq_cap) if seq_cap is not None else int(prompt_tokens_cap) + int(response_tokens_cap)
            go.seq_capacity_elems = cap
            if seq is not None:
                go.seq_prompt_col, go.seq_response_col = seq
                self.seq = payload(max(cap, 1), tdt[dock.columns[seq[0]][0]])
                go.seq = self.seq.data_ptr()
            if seq_adv:
                self.seq_advantages = payload(max(cap, 1), torch.float32)
                go.seq_advantages = self.seq_advantages.data_ptr()
        self.struct = go

    def read_result(self) -> TdResult:
        """Copies the result block to the host (synchronises the current stream)."""
        host = self.result.cpu().numpy().tobytes()
        return TdResult.from_buffer_copy(host)


class HostGetBuffers:
    """Pinned host mirrors of a GetBuffers, the destination of td_get_host."""

    def __init__(self, bufs: GetBuffers):
        import torch
        self.indices = torch.zeros(bufs.indices.shape, dtype=bufs.indices.dtype).pin_memory()
        self.cu_prompt = torch.zeros(bufs.cu_prompt.shape, dtype=torch.int32).pin_memory()
        self.cu_response = torch.zeros(bufs.cu_response.shape, dtype=torch.int32).pin_memory()
        self.cu_seq = torch.zeros(bufs.cu_seq.shape, dtype=torch.int32).pin_memory()
        self.advantages = (torch.zeros(bufs.advantages.shape, dtype=torch.float32).pin_memory()
                           if bufs.advantages is not None else None)
        # payload that the device already writes into host memory needs no second buffer
        self.payload_in_place = bool(getattr(bufs, "host_payload", False))
        self.cols = ({c: t for c, t in bufs.cols.items()} if self.payload_in_place else
                     {c: torch.zeros(t.shape, dtype=t.dtype).pin_memory() for c, t in bufs.cols.items()})
        # the result block too lives in pinned memory: a copy into pageable memory stalls the caller
        self._result_mem = torch.zeros(C.sizeof(TdResult), dtype=torch.uint8).pin_memory()
        self.result = TdResult.from_address(self._result_mem.data_ptr())
        go = TdGetOut()
        go.mode, go.pad_prompt_to, go.pad_response_to = bufs.mode, bufs.pad_prompt_to, bufs.pad_response_to
        go.flags = getattr(bufs, "flags", 0)
        go.indices, go.cu_prompt = self.indices.data_ptr(), self.cu_prompt.data_ptr()
        go.cu_response, go.cu_seq = self.cu_response.data_ptr(), self.cu_seq.data_ptr()
        for c, t in self.cols.items():
            go.col[c] = None if self.payload_in_place else t.data_ptr()      # NULL: nothing to copy
            go.col_capacity_elems[c] = t.numel()
        go.advantages = self.advantages.data_ptr() if self.advantages is not None else None
        go.result = C.addressof(self.result)
        self.struct = go

    def bytes_valid(self, dock: "Dock") -> int:
        """Bytes td_get_host copied to the host for the last call."""
        r, n = self.result, self.result.n_samples
        total = C.sizeof(TdResult) + n * 4 + 3 * (n + 1) * 4 + (n * 4 if self.advantages is not None else 0)
        for c, t in self.cols.items():
            dt, cls, _ = dock.columns[c]
            if cls == SCALAR:
                e = n
            elif self.struct.mode == PACKED:
                e = r.prompt_tokens if cls == PROMPT else r.response_tokens
            else:
                e = n * (self.struct.pad_prompt_to if cls == PROMPT else self.struct.pad_response_to)
            total += e * ELEM_SIZE[dt]
        return total


class Plan:
    """A fixed list of gets (one GetBuffers each) that td_get_many serves in one call."""

    def __init__(self, dock: "Dock", bufs: Sequence[GetBuffers], stream=None):
        import torch
        self.dock, self.bufs = dock, list(bufs)
        n = len(self.bufs)
        reqs = (TdGetReq * n)()
        for j, b in enumerate(self.bufs):
            reqs[j].consumer, reqs[j].max_samples = b.consumer, b.max_samples
            reqs[j].out = b.struct
        self.nbytes = lib().td_plan_bytes(dock.handle, n)
        self.memory = torch.empty(self.nbytes, dtype=torch.uint8, device=dock.device)
        h = C.c_void_p()
        _check("td_plan_create", lib().td_plan_create(dock.handle, reqs, n, self.memory.data_ptr(),
                                                      self.nbytes, _stream_ptr(stream), C.byref(h)))
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            lib().td_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Dock:
    """A transfer dock living in one torch-allocated workspace on `device`."""

    def __init__(self, G: int, N: int, S: int, columns: Sequence[Tuple[str, str, int]],
                 consumers: Sequence[Tuple[int, int, bool]], prompt_cap: int, response_cap: int,
                 reward_column: int, eps: float = 1e-6, device: int = 0):
        import torch
        self.G, self.N, self.S, self.n = G, N, S, G * N
        self.columns = [(DTYPE_TAG[d], CLASS_TAG[c], int(p)) for d, c, p in columns]
        self.consumers = [(int(a), int(b), bool(f)) for a, b, f in consumers]
        self.device = torch.device("cuda", device)
        self.cfg, self._keep = make_config(G, N, S, columns, consumers, prompt_cap, response_cap,
                                           reward_column, eps, device)
        self.workspace_bytes = query_workspace(self.cfg)
        self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=self.device)
        h = C.c_void_p()
        _check("td_create", lib().td_create(C.byref(self.cfg), self.workspace.data_ptr(),
                                            self.workspace_bytes, C.byref(h)))
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            lib().td_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the four calls ---------------------------------------------------
    def put(self, column: int, indices, cu, data, stream=None):
        """indices int32 [k], cu int32 [k+1] or None, data: device tensors."""
        k = indices.numel()
        _check("td_put", lib().td_put(self.handle, column, indices.data_ptr(), k,
                                      cu.data_ptr() if cu is not None else None,
                                      data.data_ptr(), data.numel(), _stream_ptr(stream)))

    def put_many(self, items, stream=None):
        """items: (column, indices, cu or None, data) device tensors, stored in this order, or
        put_items() of them."""
        arr = items if isinstance(items, C.Array) else self.put_items(items)
        _check("td_put_many", lib().td_put_many(self.handle, arr, len(arr), _stream_ptr(stream)))

    def put_back(self, bufs: GetBuffers, items: Sequence[Tuple], stream=None):
        """items: (column, data) device tensors holding the rows of the batch last served into
        `bufs`, packed in batch order; the batch size is read on the device."""
        arr = (TdBackItem * len(items))()
        for j, (column, data) in enumerate(items):
            arr[j] = TdBackItem(column, 0, data.data_ptr(), data.numel())
        _check("td_put_back", lib().td_put_back(self.handle, C.byref(bufs.struct), bufs.max_samples,
                                                arr, len(items), _stream_ptr(stream)))

    def put_back_many(self, reqs: Sequence[Tuple], stream=None):
        """reqs: (bufs, column, data): column sent back for the batch last served into bufs."""
        arr = (TdBackReq * len(reqs))()
        for j, (bufs, column, data) in enumerate(reqs):
            arr[j] = TdBackReq(C.addressof(bufs.struct), bufs.max_samples, column, data.data_ptr(), data.numel())
        _check("td_put_back_many", lib().td_put_back_many(self.handle, arr, len(reqs), _stream_ptr(stream)))

    def plan(self, bufs: Sequence[GetBuffers], stream=None) -> "Plan":
        return Plan(self, bufs, stream)

    def get_many(self, plan: "Plan", stream=None):
        _check("td_get_many", lib().td_get_many(self.handle, plan.handle, _stream_ptr(stream)))

    def get(self, bufs: GetBuffers, stream=None, max_samples: Optional[int] = None):
        _check("td_get", lib().td_get(self.handle, bufs.consumer,
                                      bufs.max_samples if max_samples is None else max_samples,
                                      C.byref(bufs.struct), _stream_ptr(stream)))

    def get_static(self, bufs: GetBuffers, stream=None):
        """The same get with the scan scratch inside the library (no scratch buffer needed;
        docks of at most 16384 prompts; calls must not overlap on the GPU)."""
        _check("td_get_static", lib().td_get_static(self.handle, bufs.consumer, bufs.max_samples,
                                                    C.byref(bufs.struct), _stream_ptr(stream)))

    def reset(self, stream=None):
        _check("td_reset", lib().td_reset(self.handle, _stream_ptr(stream)))

    def status(self, stream=None) -> TdStats:
        st = TdStats()
        _check("td_status", lib().td_status(self.handle, C.byref(st), _stream_ptr(stream)))
        return st

    # -- host-buffer variants ----------------------------------------------
    def put_host(self, column: int, indices, cu, data, stage, stream=None):
        """indices / cu / data: host tensors (pinned for asynchronous copies); stage: a device
        uint8 tensor of at least put_host_stage_bytes()."""
        k = indices.numel()
        _check("td_put_host", lib().td_put_host(self.handle, column, indices.data_ptr(), k,
                                                cu.data_ptr() if cu is not None else None,
                                                data.data_ptr(), data.numel(), stage.data_ptr(),
                                                stage.numel(), _stream_ptr(stream)))

    def put_host_stage_bytes(self, column: int, k: int, data_elems: int) -> int:
        return lib().td_put_host_stage_bytes(self.handle, column, k, data_elems)

    @staticmethod
    def put_items(items: Sequence[Tuple]):
        """The td_put_item array of (column, indices, cu or None, data) tensors, reusable across calls."""
        arr = (TdPutItem * len(items))()
        for j, (column, indices, cu, data) in enumerate(items):
            arr[j] = TdPutItem(column, indices.numel(), indices.data_ptr(),
                               cu.data_ptr() if cu is not None else None, data.data_ptr(), data.numel())
        return arr

    @staticmethod
    def host_outs(hosts: Sequence["HostGetBuffers"]):
        """The td_get_out array of a list of host mirrors, reusable across calls."""
        return (TdGetOut * len(hosts))(*[h.struct for h in hosts])

    def put_many_host(self, items, stage, stream=None):
        """items: (column, indices, cu or None, data) HOST tensors, or put_items() of them; stage:
        device uint8 tensor."""
        arr = items if isinstance(items, C.Array) else self.put_items(items)
        _check("td_put_many_host", lib().td_put_many_host(self.handle, arr, len(arr), stage.data_ptr(),
                                                          stage.numel(), _stream_ptr(stream)))

    def get_many_host(self, plan: "Plan", hosts, stage=None, stream=None):
        """hosts: HostGetBuffers per request of the plan, or host_outs() of them; stage: device
        uint8 tensor of get_many_host_stage_bytes(plan) bytes, or None."""
        arr = hosts if isinstance(hosts, C.Array) else self.host_outs(hosts)
        _check("td_get_many_host", lib().td_get_many_host(self.handle, plan.handle, arr, len(arr),
                                                          stage.data_ptr() if stage is not None else None,
                                                          stage.numel() if stage is not None else 0,
                                                          _stream_ptr(stream)))

    def get_many_host_stage_bytes(self, plan: "Plan") -> int:
        return lib().td_get_many_host_stage_bytes(plan.handle)

    def get_host(self, bufs: GetBuffers, host: "HostGetBuffers", stream=None):
        _check("td_get_host", lib().td_get_host(self.handle, bufs.consumer, bufs.max_samples,
                                                C.byref(bufs.struct), C.byref(host.struct),
                                                _stream_ptr(stream)))

    # -- measurement ------------------------------------------------------
    def kernel_timing(self, enable: bool):
        _check("td_kernel_timing", lib().td_kernel_timing(self.handle, 1 if enable else 0))

    def kernel_timing_read(self, which: int) -> Tuple[int, float]:
        n, ms = C.c_uint64(0), C.c_double(0.0)
        _check("td_kernel_timing_read", lib().td_kernel_timing_read(self.handle, which, C.byref(n), C.byref(ms)))
        return n.value, ms.value

    # -- inspection -------------------------------------------------------
    def table(self, which: int, index: int = 0):
        """Device table as a uint8 torch tensor view (copy it before the dock changes)."""
        import torch
        ptr, nbytes = C.c_void_p(), C.c_size_t()
        _check("td_debug_table", lib().td_debug_table(self.handle, which, index, C.byref(ptr), C.byref(nbytes)))
        off = ptr.value - self.workspace.data_ptr()
        return self.workspace[off:off + nbytes.value]

    def validate(self, stream=None) -> TdValidateReport:
        """Self-check of the dock's tables (synchronises the stream); report.violations == 0 if sound."""
        rep = TdValidateReport()
        _check("td_debug_validate", lib().td_debug_validate(self.handle, _stream_ptr(stream), C.byref(rep)))
        return rep

    def debug_lookback(self, poll_limit: int = 0, skip_tile: int = 0xFFFFFFFF):
        """Test hook: poll limit of the scan's look-back wait (0 = default) and a tile that withholds
        its descriptor (0xFFFFFFFF = none)."""
        _check("td_debug_lookback", lib().td_debug_lookback(self.handle, poll_limit, skip_tile))

    def launch_count(self) -> int:
        return lib().td_launch_count(self.handle)
