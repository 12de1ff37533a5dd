#!/usr/bin/env python
"""Benchmark of the transfer dock's put/get dispatch.

One step = one pass of the whole hot path over one synthetic GRPO batch: reset the dock, put
every column of every sample, then drain it for all consumers in micro-batches.  The value is
samples dispatched to consumers per second of (put phase + drain phase), with inputs resident
in HBM.  The L2 is flushed (a 256 MiB write, untimed) before each phase unless --warm-l2.

Without --config the run measures the four large shapes one after the other in one process:
the headline is the largest (the R1-shaped batch), and `per_config` carries the same record
for the 7B-, 32B- and MoE-shaped batches (the MoE shape twice: bulk, and as the scenario its
configuration describes, a producer stream against four polling consumer streams).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--sigma S] [--warm-l2]
                  [--scenario dispatch|concurrent|cascade|scan|fixed-cost] [--impl reference]
                  [--e2e-schedule pipelined|serial] [--e2e-path auto|in-place|copy]

`e2e` is the same step through the calls that take HOST buffers, bus transfers inside the timed
region; by default it is issued in two waves (the columns every worker state needs first, the
states that need nothing else served on a second stream while the other columns come in).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "td_put+td_get samples/s dispatched"
L2_FLUSH_BYTES = 256 << 20
HEADLINE_CONFIG = 5                   # the largest shape that fits one GPU
DEFAULT_CONFIGS = (5, 2, 3, 4)        # headline first
NOMINAL_HBM_GBPS = 8000.0             # the "~8 TB/s" the 70 % target is stated against
# DRAM bytes (read + write) of one launch of the copy kernels as they are built now, taken from
# the ncu summaries under profiles/: (config, kernel) -> (bytes, file, what was captured).
# A pair without a capture of the current kernels reports null.
NCU_TRAFFIC = {
    (2, "get_gather"): (80_016_128, "profiles/copy_kernels_config2_7b_shaped.md", "ncu capture of this kernel on this shape"),
    (2, "put_scatter"): (45_304_064, "profiles/copy_kernels_config2_7b_shaped.md", "ncu capture of this kernel on this shape"),
    (3, "get_gather"): (1_147_490_816, "profiles/copy_kernels_config3_32b_shaped.md", "ncu capture of this kernel on this shape"),
    (3, "put_scatter"): (733_361_920, "profiles/copy_kernels_config3_32b_shaped.md", "ncu capture of this kernel on this shape"),
}
# The larger shapes hold too much on the device for a full counter capture; their traffic is taken
# to grow with the bytes that must cross HBM, from the capture of the 32B-shaped batch:
# kernel -> (captured traffic, HBM-crossing bytes of that launch).
NCU_SCALE_FROM_CONFIG3 = {"get_gather": (1_147_490_816, 1_200_614_776), "put_scatter": (733_361_920, 784_775_700)}


def captured_traffic(cid: int, kernel: str, bytes_per_launch: float):
    """(bytes, source, note) or None."""
    if (cid, kernel) in NCU_TRAFFIC:
        return NCU_TRAFFIC[(cid, kernel)]
    if cid in (4, 5) and kernel in NCU_SCALE_FROM_CONFIG3:
        t, b = NCU_SCALE_FROM_CONFIG3[kernel]
        return (int(bytes_per_launch * t / b), "profiles/copy_kernels_config3_32b_shaped.md",
                "scaled from the capture of the 32B-shaped batch by the bytes that must cross HBM")
    return None


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=0,
                    help="workload shape 1..5; default: shapes 5 (headline), 2, 3 and 4 in one run")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-cpu-all-cores", action="store_true", help="skip the oracle-on-several-cores leg")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-variants", action="store_true", help="skip the warm-L2 and heavy-tail records")
    ap.add_argument("--e2e-path", default="auto", choices=["auto", "in-place", "copy"],
                    help="end-to-end step: where the gets leave their payload (in-place: pinned host buffers written "
                         "by the gather kernel; copy: device buffers, one transfer per column and request; auto: by size)")
    ap.add_argument("--e2e-schedule", default="pipelined", choices=["pipelined", "serial"],
                    help="end-to-end step with the batched calls: serial = one put of every column, then one "
                         "drain; pipelined = the columns every worker state needs first, the gets of the states "
                         "that need nothing else on a second stream while the other columns are still coming in")
    ap.add_argument("--api", default="many", choices=["many", "single"],
                    help="many: one td_put_many and one td_get_many per step; single: one td_put per "
                         "column and one td_get per micro-batch")
    ap.add_argument("--cpu-seconds", type=float, default=4.0, help="CPU-oracle time budget per shape and leg")
    ap.add_argument("--sigma", type=float, default=None,
                    help="spread of the lognormal response lengths (default 0.25; 0.75 is the heavy tail)")
    ap.add_argument("--warm-l2", action="store_true", help="do not flush the L2 before the phases")
    ap.add_argument("--repeat", type=int, default=10,
                    help="further passes per timed step, run right behind the timed region, for median / min / spread")
    ap.add_argument("--fused", action="store_true",
                    help="the actor update's gets also ask for the fused prompt+response id stream and "
                         "its per-token advantage twin")
    ap.add_argument("--padded", action="store_true",
                    help="gets write right-padded rows (row i at i * width, the column's pad bits behind it) "
                         "instead of packed ones; widths are the workload's maximum lengths")
    ap.add_argument("--graph", action="store_true",
                    help="cascade only: capture the step's calls into one CUDA graph once and time its replay "
                         "(nothing in the step needs the host, batch sizes are read on the device)")
    ap.add_argument("--scenario", default="dispatch", choices=["dispatch", "concurrent", "cascade", "scan", "fixed-cost"],
                    help="dispatch: put everything, then drain (the headline); concurrent: one producer stream "
                         "putting shuffled chunks of 1-64 samples while four consumer threads poll td_get on "
                         "their own streams (the out-of-order stress); cascade: generation puts in "
                         "chunks, inference states get a micro-batch and send their column back for it "
                         "(td_put_back, no host round trip), the actor update takes what is complete")
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, torch copy)"
    return 6650.0, "fallback (earlier measurement on this pool)"


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.uuid, self.proc, self.lines = uuid, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.uuid}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def count_inside(self, t_begin: float, t_end: float) -> int:
        return sum(1 for t, _ in self.lines if t_begin <= t <= t_end)

    def stop(self, t_begin: float = 0.0, t_end: float = 0.0, t_soak_end: float = 0.0):
        if self.proc:
            time.sleep(0.05)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        return self.window(t_begin, t_end, t_soak_end)

    def window(self, t_begin: float, t_end: float, t_soak_end: float = 0.0):
        """Summary of the samples taken inside [t_begin, t_end] (the timed region); when the
        region was too short to catch three, of the region and the passes behind it, else of
        everything sampled since start (all under the same load)."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        t_end = max(t_end, t_soak_end)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

        def summarise(lines):
            sm, mx, reasons = [], [], set()
            for _t, ln in lines:
                f = [x.strip() for x in ln.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for nm, val in zip(names, f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(nm)
            return sm, mx, reasons

        inside = [(t, ln) for t, ln in list(self.lines) if t_begin <= t <= t_end + 0.03]
        window = "timed region (and the passes right behind it)"
        sm, mx, reasons = summarise(inside)
        if len(sm) < 3:
            window = "everything since the start of the run"
            sm, mx, reasons = summarise(list(self.lines))
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "window": window, "reasons": sorted(reasons)}


class NvmlSampler:
    """Reads SM clock and clock-event reasons through NVML every 2 ms from a thread (read-only
    queries): nvidia-smi's own loop is too slow for a timed region of a few milliseconds."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, uuid: str):
        import pynvml
        self.nv = pynvml
        pynvml.nvmlInit()
        self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if isinstance(uuid, str) else uuid)
        self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        self.samples, self.stop_flag, self.thread = [], threading.Event(), None

    def _loop(self):
        nv = self.nv
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            nv.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self.stop_flag.is_set():
            try:
                self.samples.append((time.time(), float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)),
                                     int(get_reasons(self.h))))
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        self.thread = threading.Thread(target=self._loop, daemon=True)
        self.thread.start()

    def count_inside(self, t_begin: float, t_end: float) -> int:
        return sum(1 for s in self.samples if t_begin <= s[0] <= t_end)

    def window(self, t_begin: float, t_end: float, t_soak_end: float = 0.0):
        """Summary of the samples taken inside [t_begin, t_end]; the sampler keeps running."""
        inside = [s for s in list(self.samples) if t_begin <= s[0] <= t_end]
        window = "timed region"
        if len(inside) < 3 and t_soak_end > t_end:
            inside = [s for s in list(self.samples) if t_begin <= s[0] <= t_soak_end]
            window = "timed region and the further passes run right behind it"
        if len(inside) < 3:
            inside, window = list(self.samples), "everything since the start of the run"
        reasons = set()
        for _t, _mhz, bits in inside:
            for bit, name in self.REASONS.items():
                if bits & bit:
                    reasons.add(name)
        sm = [s[1] for s in inside]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": self.max_mhz,
                "samples": len(sm), "window": window, "source": "nvml", "reasons": sorted(reasons)}

    def stop(self, t_begin: float = 0.0, t_end: float = 0.0, t_soak_end: float = 0.0):
        self.stop_flag.set()
        if self.thread:
            self.thread.join(timeout=2)
        return self.window(t_begin, t_end, t_soak_end)


def make_sampler(torch, local_rank: int):
    gpu_id = gpu_id_for_smi(torch, local_rank)
    if gpu_id.startswith("GPU-"):
        try:
            return NvmlSampler(gpu_id)
        except Exception:
            pass
    return ClockSampler(gpu_id)


def gpu_id_for_smi(torch, local_rank: int) -> str:
    """The id nvidia-smi knows this process's device by: its UUID when listed, else its index."""
    try:
        uuid = str(torch.cuda.get_device_properties(local_rank).uuid)
        if not uuid.startswith("GPU-"):
            uuid = "GPU-" + uuid
        listed = subprocess.run(["nvidia-smi", "-L"], capture_output=True, text=True, timeout=20).stdout
        if uuid in listed:
            return uuid
    except Exception:
        pass
    return str(local_rank)


# --------------------------------------------------------------------------- multi-rank glue
def max_over_ranks(dist, values, device):
    """Element-wise maximum of `values` over all ranks (identity without a process group).
    Docks on different ranks are independent: the only exchange is this reduction of timings."""
    if dist is None:
        return list(values)
    import torch
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_rate(world: int, units_per_rank: int, seconds: float) -> float:
    """Weak scaling: every rank dispatches units_per_rank in the slowest rank's time."""
    return world * units_per_rank / seconds


# --------------------------------------------------------------------------- workload glue
def step_bytes(w, padded: bool = False, fused: bool = False):
    """Bytes one step must move, element size times true length (no alignment padding).
    put / put_ragged: every stored row read once and written once (all columns / the ragged
    ones, which are what the scatter kernel moves).  get_delivered: every delivery counted as a
    read and a write (a row that three consumers take counts three times).  get_hbm: what has to
    cross HBM when one launch serves all consumers: every stored row that anyone takes read once,
    every delivered byte written once.  In padded mode the pad writes count as bytes written."""
    from paper_2507_19017_b200 import workloads as wl
    put = sum(2 * w.data[s.name].nbytes for s in w.columns)
    put_ragged = sum(2 * w.data[s.name].nbytes for s in w.columns if s.cls != wl.SCALAR)
    written, taken = 0, set()
    for k in w.consumers:
        for name in k.out:
            spec = w.columns[w.column_index(name)]
            nbytes = w.data[name].nbytes
            if padded and spec.cls != wl.SCALAR:
                width = w.pad_prompt_to if spec.cls == wl.PROMPT else w.pad_response_to
                written += w.n * width * w.data[name].itemsize
            else:
                written += nbytes
            taken.add(name)
    read_once = sum(w.data[name].nbytes for name in taken)
    read_every = sum(w.data[name].nbytes for k in w.consumers for name in k.out)
    if fused:       # the stream: both id columns read and written once more; the twin: one float written per token
        extra = w.data["prompt_ids"].nbytes + w.data["response_ids"].nbytes
        read_every += extra
        written += extra + 4 * w.tokens_total()
    return {"put": put, "put_ragged": put_ragged, "get_delivered": read_every + written,
            "get_hbm": read_once + written}


class GpuStep:
    """Device-resident inputs and per-get output buffers of one step, and the step itself."""

    def __init__(self, w, device_index: int, api: str = "many", fused: bool = False, padded: bool = False,
                 warm_l2: bool = False):
        import torch
        self.api = api
        self.warm_l2 = warm_l2
        self.e2e_path = "auto"
        self.e2e_schedule = "pipelined"
        self.e2e_waves = None
        from paper_2507_19017_b200 import binding as td
        from paper_2507_19017_b200 import workloads as wl
        self.torch, self.td, self.w = torch, td, w
        torch.cuda.set_device(device_index)
        self.dev = torch.device("cuda", device_index)
        self.dock = td.Dock(w.G, w.N, w.S, w.column_tuples(), w.consumer_tuples(),
                            w.shard_capacity(wl.PROMPT), w.shard_capacity(wl.RESPONSE),
                            w.column_index("reward"), 1e-6, device_index)
        self.puts = []        # (column, idx, cu, data) device tensors
        self.host_puts = []   # the same in pinned host memory
        self.h2d_bytes = 0
        # A worker that sends a whole record has one index array for the batch and one cu array
        # per length class: columns with equal arrays share them, on the host and on the device.
        shared = {}
        counted = set()

        def share(a):
            key = (a.dtype.str, a.shape, a.tobytes())
            if key not in shared:
                pinned = self._pin(a)
                shared[key] = (pinned, pinned.to(self.dev))
            return shared[key]

        for op in w.ops:
            if op.kind != "put":
                continue
            cu, data = w.pack(op.column, op.indices)
            idx = np.ascontiguousarray(op.indices, dtype=np.int32)
            h_idx, d_idx = share(idx)
            h_cu, d_cu = share(cu) if cu is not None else (None, None)
            h_data = self._pin(data)
            self.host_puts.append((op.column, h_idx, h_cu, h_data))
            self.puts.append((op.column, d_idx, d_cu, h_data.to(self.dev)))
            # the batched host call brings a shared array over once, the per-column call every time
            for h, arr in ((h_idx, idx), (h_cu, cu)):
                if arr is not None and not (api == "many" and h.data_ptr() in counted):
                    self.h2d_bytes += arr.nbytes
                    counted.add(h.data_ptr())
            self.h2d_bytes += data.nbytes
        # one output buffer set per get call, sized by the longest rows it could meet
        lp = np.sort(w.len_prompt)[::-1]
        lr = np.sort(w.len_response)[::-1]
        self.gets = []
        for op in w.ops:
            if op.kind != "get":
                continue
            m = op.max_samples
            stream = fused and w.consumers[op.consumer].advantage
            bufs = td.GetBuffers(self.dock, op.consumer, m, td.PADDED if padded else td.PACKED,
                                 w.pad_prompt_to if padded else 0, w.pad_response_to if padded else 0,
                                 prompt_tokens_cap=int(lp[:m].sum(dtype=np.int64)),
                                 response_tokens_cap=int(lr[:m].sum(dtype=np.int64)),
                                 seq=(w.column_index("prompt_ids"), w.column_index("response_ids")) if stream else None,
                                 seq_adv=stream)
            self.gets.append(bufs)
        self.plan = self.dock.plan(self.gets) if api == "many" else None
        self.flush_buf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=self.dev)
        self.stage = None
        self.host_gets = None

    def _pin(self, a):
        t = self.torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else np.ascontiguousarray(a))
        if a.dtype == np.uint16:
            t = t.view(self.torch.bfloat16)
        return t.pin_memory()

    def flush_l2(self):
        """Ahead of a timed phase: the 256 MiB write that empties L2, or (warm variant) a spin of
        about 100 us that touches no memory.  Either keeps the device busy while the host
        enqueues the phase's launches, so that the events time the device, not the host."""
        if not self.warm_l2:
            self.flush_buf.zero_()
        else:
            self.torch.cuda._sleep(200_000)

    def close(self):
        """Gives the device memory back (the next shape of the run needs it)."""
        if self.plan is not None:
            self.plan.close()
        self.dock.close()
        for name in ("puts", "host_puts", "gets", "plan", "flush_buf", "stage", "host_gets", "meta_stage",
                     "host_put_arr", "host_out_arr", "e2e_gets", "e2e_plan", "dock"):
            if hasattr(self, name):
                setattr(self, name, None)
        self.torch.cuda.empty_cache()

    def put_phase(self):
        self.dock.reset()
        if self.api == "many":
            self.dock.put_many(self.puts)
        else:
            for col, idx, cu, data in self.puts:
                self.dock.put(col, idx, cu, data)

    def drain_phase(self):
        if self.api == "many":
            self.dock.get_many(self.plan)
        else:
            for bufs in self.gets:
                self.dock.get(bufs)

    def timed_step(self):
        """Returns (put_ms, drain_ms) measured with CUDA events on the current stream."""
        torch = self.torch
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        self.flush_l2()
        ev[0].record(); self.put_phase(); ev[1].record()
        self.flush_l2()
        ev[2].record(); self.drain_phase(); ev[3].record()
        torch.cuda.synchronize()
        return ev[0].elapsed_time(ev[1]), ev[2].elapsed_time(ev[3])

    def served(self):
        """Samples and tokens the last drain dispatched (reads the result blocks)."""
        s = t = 0
        for bufs in self.gets:
            r = bufs.read_result()
            s += r.n_samples
            t += r.prompt_tokens + r.response_tokens
        return s, t

    # end to end: host buffers in, host buffers out
    def prepare_e2e(self):
        """Host-side state of the end-to-end step.  Batched form: the inputs are pinned host
        arrays that td_put_many_host brings over; the gets of a second plan write their payload
        straight into pinned host buffers (the device addresses them), and td_get_many_host
        fetches every request's result block, indices, cu_seqlens and advantages in one transfer."""
        td, torch = self.td, self.torch
        needs = [self.dock.put_host_stage_bytes(c, i.numel(), d.numel()) for c, i, _cu, d in self.host_puts]
        if self.api == "many":
            self.stage = [torch.empty(sum(needs), dtype=torch.uint8, device=self.dev)]
            # Where the device leaves the payload: many small columns (a few hundred KB each) are
            # written into pinned host buffers by the gather kernel itself, which costs no call per
            # piece; large ones go to device buffers and come over with one copy-engine transfer
            # each, which moves a long piece a little faster than the kernel's stores do.
            w = self.w
            out_bytes = sum(w.data[name].nbytes for k in w.consumers for name in k.out)
            pieces = sum(len(b.cols) for b in self.gets)
            self.e2e_in_place = (out_bytes / max(pieces, 1) < (2 << 20)) if self.e2e_path == "auto" else self.e2e_path == "in-place"
            self.e2e_gets = ([td.GetBuffers(self.dock, b.consumer, b.max_samples, b.mode, b.pad_prompt_to, b.pad_response_to,
                                            capacities=dict(b.caps), host_payload=True) for b in self.gets]
                             if self.e2e_in_place else self.gets)
            self.e2e_plan = self.dock.plan(self.e2e_gets) if self.e2e_in_place else self.plan
            self.host_gets = [td.HostGetBuffers(b) for b in self.e2e_gets]
            self.meta_stage = torch.empty(self.dock.get_many_host_stage_bytes(self.e2e_plan), dtype=torch.uint8, device=self.dev)
            # Pipelined schedule: the columns that every worker state needs go first; the states
            # that need nothing else are served on a second stream as soon as those are stored,
            # while the remaining columns are still crossing the bus in the other direction.
            need = [set(w.column_index(nm) for nm in k.need) for k in w.consumers]
            first_cols = set.intersection(*need)
            early = {c for c, nd in enumerate(need) if nd <= first_cols}
            self.e2e_waves = None
            if self.e2e_schedule == "pipelined" and early and len(early) < len(need) and first_cols:
                waves = []
                for cols, cons in ((first_cols, early), (None, set(range(len(need))) - early)):
                    puts = [p for p in self.host_puts if (p[0] in first_cols) == (cols is not None)]
                    gets = [b for b in self.e2e_gets if b.consumer in cons]
                    hosts = [h for b, h in zip(self.e2e_gets, self.host_gets) if b.consumer in cons]
                    plan = self.dock.plan(gets)
                    waves.append({
                        "put_arr": self.dock.put_items(puts),
                        "stage": torch.empty(sum(self.dock.put_host_stage_bytes(c, i.numel(), d.numel()) for c, i, _cu, d in puts),
                                             dtype=torch.uint8, device=self.dev),
                        "plan": plan, "out_arr": self.dock.host_outs(hosts),
                        "meta": torch.empty(self.dock.get_many_host_stage_bytes(plan), dtype=torch.uint8, device=self.dev),
                        "h2d": sum(d.numel() * d.element_size() for _c, _i, _cu, d in puts)
                               + sum(t.numel() * 4 for t in {id(x): x for _c, i, cu, _d in puts for x in (i, cu) if x is not None}.values()),
                        "h2d_copies": len(puts) + len({x.data_ptr() for _c, i, cu, _d in puts for x in (i, cu) if x is not None}),
                        "d2h_copies": sum(len(b.cols) for b in gets)})
                self.e2e_waves = waves
                self.e2e_stream = torch.cuda.Stream(device=self.dev)
                self.e2e_event = torch.cuda.Event()
        else:
            self.stage = [torch.empty(max(needs), dtype=torch.uint8, device=self.dev) for _ in range(2)]
            self.host_gets = [td.HostGetBuffers(b) for b in self.gets]
        self.host_put_arr = self.dock.put_items(self.host_puts)       # marshalled once, like a caller would
        self.host_out_arr = self.dock.host_outs(self.host_gets)

    def e2e_step(self):
        torch = self.torch
        self.dock.reset()
        if self.api == "many" and self.e2e_waves:
            a, b = self.e2e_waves
            self.dock.put_many_host(a["put_arr"], a["stage"])
            self.e2e_event.record()
            self.dock.put_many_host(b["put_arr"], b["stage"])                  # on its way while the first states are served
            self.e2e_stream.wait_event(self.e2e_event)
            self.dock.get_many_host(a["plan"], a["out_arr"], a["meta"], stream=self.e2e_stream)
            self.dock.get_many_host(b["plan"], b["out_arr"], b["meta"])
            return None
        if self.api == "many":          # one call in, one call out: two synchronisations per step
            self.dock.put_many_host(self.host_put_arr, self.stage[0])
            self.dock.get_many_host(self.e2e_plan, self.host_out_arr, self.meta_stage)
            return None
        for j, (col, idx, cu, data) in enumerate(self.host_puts):
            if j >= 2:
                self.stage_ev[j % 2].synchronize()      # staging buffer free again
            self.dock.put_host(col, idx, cu, data, self.stage[j % 2])
            self.stage_ev[j % 2].record()
        for bufs, host in zip(self.gets, self.host_gets):
            self.dock.get_host(bufs, host)
        torch.cuda.synchronize()
        return None

    def run_e2e(self, steps: int, warmup: int):
        torch = self.torch
        self.prepare_e2e()
        self.stage_ev = [torch.cuda.Event() for _ in range(2)]
        for _ in range(warmup):
            self.e2e_step()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(steps):
            self.e2e_step()
        torch.cuda.synchronize()
        el = (time.perf_counter() - t0) / steps
        served = sum(h.result.n_samples for h in self.host_gets)
        assert served == self.w.n * len(self.w.consumers), f"end-to-end drain served {served} samples"
        d2h = sum(h.bytes_valid(self.dock) for h in self.host_gets)      # counted from what the last step brought over
        if self.api == "many" and self.e2e_waves:
            self.e2e_h2d_bytes = sum(wv["h2d"] for wv in self.e2e_waves)
            copies = {"h2d_copies_per_step": sum(wv["h2d_copies"] for wv in self.e2e_waves),
                      "d2h_copies_per_step": 2 if self.e2e_in_place else 2 + sum(wv["d2h_copies"] for wv in self.e2e_waves),
                      "d2h_path": ("payload written into pinned host buffers by the gather kernel" if self.e2e_in_place else
                                   "one transfer per served column and request from device buffers") +
                                  "; one more transfer per wave for all its result blocks, indices, cu_seqlens and advantages",
                      "schedule": "two waves: td_put_many_host of the columns every worker state needs, then of the "
                                  "rest, on one stream; td_get_many_host for the states that need only the first "
                                  "columns on a second stream behind the first put (its transfers to the host run "
                                  "while the second put's come in), then td_get_many_host for the other states"}
            for wv in self.e2e_waves:
                wv["plan"].close()
            self.e2e_waves = None
        elif self.api == "many":
            shared = len({h.data_ptr() for _c, h, _cu, _d in self.host_puts}) + \
                len({cu.data_ptr() for _c, _h, cu, _d in self.host_puts if cu is not None})
            if self.e2e_in_place:
                copies = {"h2d_copies_per_step": shared + len(self.host_puts), "d2h_copies_per_step": 1,
                          "d2h_path": "payload written into pinned host buffers by the gather kernel; one transfer "
                                      "for all result blocks, indices, cu_seqlens and advantages"}
            else:
                copies = {"h2d_copies_per_step": shared + len(self.host_puts),
                          "d2h_copies_per_step": 1 + sum(len(b.cols) for b in self.gets),
                          "d2h_path": "one transfer per served column and request from device buffers; one more "
                                      "for all result blocks, indices, cu_seqlens and advantages"}
        else:
            copies = {"h2d_copies_per_step": sum(2 + (cu is not None) for _c, _h, cu, _d in self.host_puts),
                      "d2h_copies_per_step": None, "d2h_path": "one transfer per array and request"}
        if getattr(self, "e2e_plan", None) is not None and self.e2e_plan is not self.plan:
            self.e2e_plan.close()
        self.e2e_plan = self.e2e_gets = None
        return el, d2h, copies


class CascadeStep:
    """The whole sample flow as one step: the schedule's generation puts, gets and write-backs
    enqueued in order on one stream with no host synchronisation in between.  Each consumer
    reuses one set of output buffers (a worker state has used its batch up by the time it asks
    for the next)."""

    def __init__(self, w, device_index: int):
        import torch
        from paper_2507_19017_b200 import binding as td
        from paper_2507_19017_b200 import workloads as wl
        self.torch, self.td, self.w = torch, td, w
        torch.cuda.set_device(device_index)
        self.dev = torch.device("cuda", device_index)
        self.dock = td.Dock(w.G, w.N, w.S, w.column_tuples(), w.consumer_tuples(),
                            w.shard_capacity(wl.PROMPT), w.shard_capacity(wl.RESPONSE),
                            w.column_index("reward"), 1e-6, device_index)

        def dev(a):
            t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else np.ascontiguousarray(a))
            return (t.view(torch.bfloat16) if a.dtype == np.uint16 else t).to(self.dev)

        lp = np.sort(w.len_prompt)[::-1]
        lr = np.sort(w.len_response)[::-1]
        m = w.micro_batch
        self.bufs = [td.GetBuffers(self.dock, c, m, td.PACKED, prompt_tokens_cap=int(lp[:m].sum(dtype=np.int64)),
                                   response_tokens_cap=int(lr[:m].sum(dtype=np.int64)))
                     for c in range(len(w.consumers))]
        pool = {c: dev(a) for c, a in w.pool.items()}
        self.plans = {}
        self.graph = None
        self.calls = []
        self.put_bytes = 0
        for op in w.ops:
            if op.kind == "put":
                cu, data = w.pack(op.column, op.indices)
                self.calls.append(("put", op.column, dev(np.ascontiguousarray(op.indices, np.int32)),
                                   dev(cu) if cu is not None else None, dev(data)))
                self.put_bytes += 2 * data.nbytes
            elif op.kind == "get":
                self.calls.append(("get", self.bufs[op.consumer]))
            elif op.kind == "get_many":
                key = tuple(op.group)
                if key not in self.plans:
                    self.plans[key] = self.dock.plan([self.bufs[c] for c in op.group])
                self.calls.append(("get_many", self.plans[key]))
            elif op.kind == "put_back_many":
                self.calls.append(("back_many", [(self.bufs[c], col, pool[col]) for c, col in op.group]))
            else:
                self.calls.append(("back", self.bufs[op.consumer], [(c, pool[c]) for c in op.columns]))
        self.flush_buf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=self.dev)
        # per-consumer totals are accumulated on the device from the result blocks
        self.served_acc = torch.zeros(2, dtype=torch.int64, device=self.dev)

    def run(self):
        d = self.dock
        d.reset()
        for call in self.calls:
            if call[0] == "put":
                d.put(call[1], call[2], call[3], call[4])
            elif call[0] == "get":
                d.get(call[1])
            elif call[0] == "get_many":
                d.get_many(call[1])
            elif call[0] == "back_many":
                d.put_back_many(call[1])
            else:
                d.put_back(call[1], call[2])

    def capture(self):
        """Records the step's calls into a CUDA graph; timed_step then replays it."""
        torch = self.torch
        self.run()
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self.run()
        torch.cuda.synchronize()

    def timed_step(self):
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.flush_buf.zero_()
        e0.record()
        if self.graph is not None:
            self.graph.replay()
        else:
            self.run()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    def served(self):
        st = self.dock.status()
        n_c = len(self.w.consumers)
        return sum(st.got_samples[c] for c in range(n_c)), sum(st.got_tokens[c] for c in range(n_c))

    def written_back(self):
        st = self.dock.status()
        return {self.w.columns[c].name: int(st.put_accepted[c]) for c in self.w.pool}


def run_fixed_cost(args, local_rank):
    """What a put phase and a drain cost before any byte moves: the 7B-shaped dock (2048 samples,
    128 requests of 64) with every row length divided by 64, 16, 4, 2 and 1, and the same rows
    in docks of 64 to 8192 samples.  Prints one JSON line with the times and, for the first
    series, the straight line time = fixed + bytes / rate fitted through them."""
    import torch
    from paper_2507_19017_b200 import workloads as wl
    peak, peak_kind = load_peaks()
    reps = max(2 * args.steps, 20)

    def timed(w):
        step = GpuStep(w, local_rank)
        for _ in range(5):
            step.timed_step()
        t = [step.timed_step() for _ in range(reps)]
        sb = step_bytes(w)
        put_b, drain_b = sb["put"], sb["get_hbm"]
        step.close()
        return statistics.mean(x[0] for x in t) * 1e3, statistics.mean(x[1] for x in t) * 1e3, put_b, drain_b

    by_length = []
    for scale in (64, 16, 4, 2, 1):
        w = wl.make_custom(f"7b-shaped-rows-1/{scale}", 256, 8, 4, prompt_len=(max(128 // scale, 1), max(1024 // scale, 2)),
                           response=("lognormal", 1500.0 / scale, wl.SIGMA_HEADLINE, max(4096 // scale, 4)),
                           vocab=152064, micro_batch=64, seed=wl.BASE_SEED, schedule="bulk", config_id=2)
        put_us, drain_us, put_b, drain_b = timed(w)
        by_length.append({"row_length_scale": f"1/{scale}", "put_us": put_us, "drain_us": drain_us,
                          "put_hbm_bytes": put_b, "drain_hbm_bytes": drain_b})
    fit = {}
    for ph in ("put", "drain"):
        x = np.array([r[f"{ph}_hbm_bytes"] for r in by_length], dtype=np.float64)
        y = np.array([r[f"{ph}_us"] for r in by_length], dtype=np.float64)
        slope, fixed = np.polyfit(x, y, 1)
        fit[ph] = {"fixed_us": float(fixed), "GBps_of_the_rest": float(1e-3 / slope) if slope > 0 else None,
                   "frac_of_measured_copy": float(1e-3 / slope / peak) if slope > 0 else None}
    by_samples = []
    for G, mb in ((8, 64), (32, 64), (128, 64), (256, 64), (1024, 64)):
        w = wl.make_custom(f"short-rows-{G * 8}", G, 8, 4, prompt_len=(2, 16), response=("lognormal", 24.0, wl.SIGMA_HEADLINE, 64),
                           vocab=152064, micro_batch=mb, seed=wl.BASE_SEED, schedule="bulk", config_id=2)
        put_us, drain_us, _pb, _db = timed(w)
        by_samples.append({"samples": w.n, "requests": 4 * (w.n // mb), "put_us": put_us, "drain_us": drain_us})
    print(json.dumps({"scenario": "fixed-cost", "api": "td_put_many + td_get_many (3 + 3 launches per step)",
                      "l2": "flushed before each phase (256 MiB write)", "timed_steps_per_point": reps,
                      "by_row_length": by_length, "fit_time_us_equals_fixed_plus_bytes_over_rate": fit,
                      "by_samples_with_rows_of_a_few_tokens": by_samples, "peak_GBps": peak, "peak_kind": peak_kind}))


def run_scan(args, local_rank):
    """Readiness scan at sizes where bytes, not latency, bound it: docks of 2^20 .. 2^24 samples
    that hold only the scalar reward, one consumer that needs just that.  Times a get of one
    micro-batch (every group's status words are read, the lowest ready groups are served) with
    every sample ready and with none ready, and prints one JSON line."""
    import torch
    from paper_2507_19017_b200 import binding as td
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peak, peak_kind = load_peaks()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    N = 16
    rows = []
    for log_n in (20, 22, 24):
        n = 1 << log_n
        G = n // N
        dock = td.Dock(G, N, 16, [("i32", "prompt", 0), ("i32", "response", 0), ("f32", "scalar", 0)],
                       [(4, 4, True)], 64, 64, 2, 1e-6, local_rank)
        idx = torch.arange(n, dtype=torch.int32, device=dev)
        rew = torch.randn(n, dtype=torch.float32, device=dev)
        bufs = td.GetBuffers(dock, 0, 128, td.PACKED, prompt_tokens_cap=8, response_tokens_cap=8)

        def timed_get():
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            flush.zero_()
            e0.record(); dock.get(bufs); e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1)

        empty = min(timed_get() for _ in range(max(args.warmup, 3) + 5))
        assert bufs.read_result().n_samples == 0
        dock.put(2, idx, None, rew)
        ready, served = [], 0
        for _ in range(max(args.warmup, 3) + 5):
            ready.append(timed_get())
            r = bufs.read_result()
            assert r.n_samples == 128 and r.status == 0
            served += r.n_samples
        scan_bytes = n * 4 + G // 8                     # status words + claim bits
        rows.append({"samples": n, "groups": G, "tiles": -(-G // (256 * (4 if G > 65536 else 1))), "status_MB": scan_bytes / 1e6,
                     "get_us_none_ready": empty * 1e3, "get_us_all_ready": min(ready) * 1e3,
                     "scan_GBps_all_ready": scan_bytes / (min(ready) * 1e-3) / 1e9,
                     "frac_of_peak": scan_bytes / (min(ready) * 1e-3) / 1e9 / peak})
        assert dock.status().error_word == 0
        dock.close()
        del dock, idx, rew, bufs
        torch.cuda.empty_cache()
    print(json.dumps({"metric": "td_get readiness scan", "unit": "us per get of 128 samples (select + finalize + gather)",
                      "peak_GBps": peak, "peak_kind": peak_kind, "l2": "flushed before each get", "sizes": rows}))


def run_cascade(args, w, local_rank, world, dist, config):
    """Times the cascade scenario and prints its JSON line (rank 0)."""
    import torch
    step = CascadeStep(w, local_rank)
    launches_one_step = None
    if args.graph:
        n0 = step.dock.launch_count()
        step.capture()
        launches_one_step = (step.dock.launch_count() - n0) // 2      # run once eagerly, once under capture
    peak, peak_kind = load_peaks()
    sampler = make_sampler(torch, local_rank)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step.timed_step()
    served_s, served_t = step.served()
    n_dispatch = w.n * len(w.consumers)
    assert served_s == n_dispatch, f"cascade served {served_s} of {n_dispatch} samples"
    back = step.written_back()
    assert all(v == w.n for v in back.values()), back
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    t_begin = time.time()
    torch.cuda.cudart().cudaProfilerStart()
    launches0 = step.dock.launch_count()
    ms = [step.timed_step() for _ in range(args.steps)]
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    torch.cuda.cudart().cudaProfilerStop()
    t_end = time.time()
    launches = step.dock.launch_count() - launches0
    if launches_one_step is not None:
        launches = launches_one_step * args.steps          # replayed from the graph
    clocks = sampler.stop(t_begin, t_end)
    ms_per_step, = max_over_ranks(dist, [sum(ms) / len(ms)], step.dev)
    peak_nominal = NOMINAL_HBM_GBPS
    graph, step.graph = step.graph, None                    # the per-kernel pass below runs eagerly
    # algorithmic bytes: every stored row read and written once, every served row read and written once
    sb = step_bytes(w)
    get_bytes, put_bytes = sb["get_delivered"], sb["put"]
    step.dock.kernel_timing(True)
    ksteps = min(args.steps, 3)
    for _ in range(ksteps):
        step.timed_step()
    n_sc, ms_sc = step.dock.kernel_timing_read(0)
    n_ga, ms_ga = step.dock.kernel_timing_read(1)
    step.dock.kernel_timing(False)
    ragged_put = sum(2 * w.data[s.name].nbytes for s in w.columns if s.cls != "scalar")
    kern = {"put_scatter": {"launches_per_step": n_sc // ksteps, "avg_ms": ms_sc / max(n_sc, 1),
                            "bytes_per_launch": ragged_put / max(n_sc // ksteps, 1)},
            "get_gather": {"launches_per_step": n_ga // ksteps, "avg_ms": ms_ga / max(n_ga, 1),
                           "bytes_per_launch": get_bytes / max(n_ga // ksteps, 1)}}
    for k in kern.values():
        k["GBps"] = k["bytes_per_launch"] / (k["avg_ms"] * 1e-3) / 1e9 if k["avg_ms"] > 0 else 0.0
    dom = "get_gather" if ms_ga >= ms_sc else "put_scatter"
    if int(os.environ.get("RANK", "0")) != 0:
        return
    calls = {k: sum(1 for c in step.calls if c[0] == k) for k in ("put", "get", "back", "get_many", "back_many")}
    calls = {k: v for k, v in calls.items() if v}
    line = {
        "metric": METRIC, "value": whole_job_rate(world, n_dispatch, ms_per_step * 1e-3), "unit": "samples/s",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": dict(config, scenario="cascade", calls_per_step=calls,
                       launch="one CUDA graph replay per step" if graph is not None else "eager calls",
                       api=("td_put per generation chunk, one td_get_many + one td_put_back_many per poll of all "
                            "worker states, one stream, no host sync" if args.api == "many" else
                            "td_put per generation chunk, td_get + td_put_back per micro-batch, one stream, no host sync"),
                       l2="flushed before each step (256 MiB write)"),
        "tokens_per_s": world * served_t / (ms_per_step * 1e-3),
        "step_GBps": (put_bytes + get_bytes) / (ms_per_step * 1e-3) / 1e9,
        "kernels": kern,
        "roofline": {"bound": "latency", "kernel": dom, "achieved": kern[dom]["GBps"], "peak": peak, "unit": "GB/s",
                     "frac": kern[dom]["GBps"] / peak, "frac_of_nominal_8TBps": kern[dom]["GBps"] / peak_nominal,
                     "traffic": None, "traffic_source": None, "peak_kind": peak_kind,
                     "bytes_per_launch": kern[dom]["bytes_per_launch"], "avg_launch_ms": kern[dom]["avg_ms"],
                     "note": "average over many small launches, every delivery counted as read + write: this "
                             "scenario is bound by launch latency"},
        "cpu_baseline": None, "e2e": None,
        "gpu_launches": launches, "gpu_launches_per_step": launches // args.steps, "clocks": clocks,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- CPU oracle
def time_oracle(w, budget_s: float, steps: int = 0, warmup: int = 0):
    """The oracle as it stands, one thread, whole steps of the same workload.  steps = 0: as many
    as fit the time budget (at least one); else `warmup` untimed steps and `steps` timed ones,
    cut short when six times the budget is used up.  One set of output buffers per consumer.
    Returns (samples/s, steps timed, seconds)."""
    from oracle import td_oracle as ora
    from paper_2507_19017_b200 import workloads as wl
    d = ora.OracleDock(w.G, w.N, w.S, w.column_tuples(), w.consumer_tuples(),
                       w.shard_capacity(wl.PROMPT), w.shard_capacity(wl.RESPONSE),
                       w.column_index("reward"), 1e-6)
    puts = []
    for op in w.ops:
        if op.kind == "put":
            cu, data = w.pack(op.column, op.indices)
            puts.append((op.column, np.ascontiguousarray(op.indices, dtype=np.int32), cu, np.ascontiguousarray(data)))
    lp = np.sort(w.len_prompt)[::-1]
    lr = np.sort(w.len_response)[::-1]
    prepared = {}
    gets = []
    for op in w.ops:
        if op.kind == "get":
            key = (op.consumer, op.max_samples)
            if key not in prepared:
                m = op.max_samples
                caps = {}
                for c, (dt, cls, _p) in enumerate(d.columns):
                    caps[c] = m if cls == 0 else int((lp if cls == 1 else lr)[:m].sum(dtype=np.int64))
                prepared[key] = d.prepare_get(op.consumer, m, caps)
            gets.append(prepared[key])

    def one_step():
        d.reset()
        for col, idx, cu, data in puts:
            d.put_raw(col, idx, cu, data)
        return sum(d.get_prepared(g) for g in gets)

    t_start = time.perf_counter()
    for _ in range(warmup if steps else 0):
        one_step()
        if time.perf_counter() - t_start > budget_s:
            break
    done, samples = 0, 0
    t0 = time.perf_counter()
    while True:
        samples += one_step()
        done += 1
        el = time.perf_counter() - t0
        if (steps and done >= steps) or (not steps and el >= budget_s) or el >= 6.0 * budget_s:
            break
    d.close()
    return samples / el, done, el


def _oracle_worker(args):
    """One host process of the all-cores leg: its own copy of the workload and of the oracle."""
    cid, sigma, budget = args
    from oracle import td_oracle
    td_oracle.build()
    w = make_workload(cid, 0, sigma, "bulk")
    return time_oracle(w, budget)


def time_oracle_all_cores(cid: int, sigma, budget_s: float, max_workers: int = 8):
    """The same oracle, unchanged, on several host cores at once: one process per core, each with
    its own dock over the same workload (the oracle is one thread by design; this is what the
    host can dispatch when every core runs one).  Processes are spawned, not forked.  Returns
    (samples/s summed over the processes, processes, seconds of the slowest)."""
    import multiprocessing as mp
    workers = max(1, min(os.cpu_count() or 1, max_workers))
    with mp.get_context("spawn").Pool(workers) as pool:
        res = pool.map(_oracle_worker, [(cid, sigma, budget_s)] * workers)
    return sum(r[0] for r in res), workers, max(r[2] for r in res)


# --------------------------------------------------------------------------- one shape, measured
def make_workload(cid: int, rank: int, sigma, schedule: str):
    from paper_2507_19017_b200 import workloads as wl
    return wl.make_config(cid, seed=wl.BASE_SEED + cid + 1000 * rank,
                          sigma=wl.SIGMA_HEADLINE if sigma is None else sigma, schedule=schedule)


def config_dict(w, cid: int, sigma, warm_l2: bool):
    from paper_2507_19017_b200 import workloads as wl
    return {"workload": f"configs[{cid - 1}] {w.name}", "G": w.G, "N": w.N, "S": w.S,
            "samples": w.n, "tokens": w.tokens_total(), "micro_batch": w.micro_batch,
            "consumers": len(w.consumers), "schedule": "one put per column, then round-robin gets",
            "l2": "warm (not flushed)" if warm_l2 else "flushed before each phase (256 MiB write)",
            "response_sigma": wl.SIGMA_HEADLINE if sigma is None else sigma}


def kernel_record(ms_total: float, launches: int, passes: int, hbm_bytes: float, delivered_bytes: float, peak: float):
    per = max(launches // max(passes, 1), 1)
    avg = ms_total / max(launches, 1)
    rec = {"launches_per_step": launches // max(passes, 1), "avg_ms": avg,
           "bytes_per_launch": hbm_bytes / per, "delivered_bytes_per_launch": delivered_bytes / per}
    rec["GBps"] = rec["bytes_per_launch"] / (avg * 1e-3) / 1e9 if avg > 0 else 0.0
    rec["delivered_GBps"] = rec["delivered_bytes_per_launch"] / (avg * 1e-3) / 1e9 if avg > 0 else 0.0
    rec["frac_of_measured_copy"] = rec["GBps"] / peak
    rec["frac_of_nominal_8TBps"] = rec["GBps"] / NOMINAL_HBM_GBPS
    return rec


def measure_steps(step, steps: int, warmup: int, repeat: int, dist, sampler):
    """Warm-up, then exactly `steps` timed steps between barriers, then further passes for the
    spread.  Returns the timings and the clock record of that window."""
    torch = step.torch

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(warmup, 3)):
        step.timed_step()
    barrier()
    t_begin = time.time()
    torch.cuda.cudart().cudaProfilerStart()        # lets a profiler capture the timed region only
    launches0 = step.dock.launch_count()
    put_ms, drain_ms = [], []
    for _ in range(steps):
        a, b = step.timed_step()
        put_ms.append(a); drain_ms.append(b)
    barrier()
    torch.cuda.cudart().cudaProfilerStop()
    t_end = time.time()
    launches = step.dock.launch_count() - launches0
    # further passes right behind the timed region: the spread of a step, and clock samples under
    # the same load when the region itself lasted only a few milliseconds
    extra = []
    budget = time.time() + 2.0
    while len(extra) < min(repeat * steps, 400) and time.time() < budget:
        a, b = step.timed_step()
        extra.append(a + b)
    while time.time() - t_end < 0.25 and sampler.count_inside(t_begin, time.time()) < 8:
        a, b = step.timed_step()
        extra.append(a + b)
    t_soak_end = time.time()
    clocks = sampler.window(t_begin, t_end, t_soak_end)
    allp = [a + b for a, b in zip(put_ms, drain_ms)] + extra
    spread = {"passes": len(allp), "median_ms": statistics.median(allp), "min_ms": min(allp), "max_ms": max(allp),
              "note": f"the {steps} timed steps and {len(extra)} further passes run right behind them"}
    return put_ms, drain_ms, launches, clocks, spread


def measure_dispatch(args, cid: int, rank: int, local_rank: int, world: int, dist, sampler, *, sigma=None,
                     warm_l2: bool = False, with_e2e: bool = True, with_cpu: bool = True, brief: bool = False):
    """The record of one shape: step time, phases, the two copy kernels, roofline, end to end, CPU
    oracle.  brief: a variant record (no per-kernel pass, no e2e, no CPU leg, few steps)."""
    import torch
    w = make_workload(cid, rank, sigma, "bulk")
    config = config_dict(w, cid, sigma, warm_l2)
    n_dispatch = w.n * len(w.consumers)
    step = GpuStep(w, local_rank, args.api, args.fused, args.padded, warm_l2)
    step.e2e_path = args.e2e_path
    step.e2e_schedule = args.e2e_schedule
    if args.padded:
        config["output"] = f"right-padded rows, widths {w.pad_prompt_to} / {w.pad_response_to}"
    if args.fused:
        config["fused_stream"] = "actor-update gets also write the prompt+response id stream and its advantage twin"
    peak, peak_kind = load_peaks()
    sb = step_bytes(w, args.padded, args.fused)
    steps = max(min(args.steps, 5), 1) if brief else args.steps
    put_ms, drain_ms, launches, clocks, spread = measure_steps(step, steps, args.warmup, 2 if brief else args.repeat,
                                                               dist, sampler)
    served_s, served_t = step.served()
    assert served_s == n_dispatch, f"drain served {served_s} of {n_dispatch} samples"
    mean_put, mean_drain = sum(put_ms) / len(put_ms), sum(drain_ms) / len(drain_ms)
    ms_per_step = mean_put + mean_drain
    ms_per_step, mean_put, mean_drain = max_over_ranks(dist, [ms_per_step, mean_put, mean_drain], step.dev)
    rec = {
        "config": config, "api": ("td_put_many + td_get_many (one call each per step)" if args.api == "many"
                                  else "td_put per column + td_get per micro-batch"),
        "value": whole_job_rate(world, n_dispatch, ms_per_step * 1e-3), "unit": "samples/s",
        "ms_per_step": ms_per_step, "ms_per_step_median": spread["median_ms"], "ms_per_step_min": spread["min_ms"],
        "spread": spread,
        "tokens_per_s": world * served_t / (ms_per_step * 1e-3),
        "phases": {"put_ms": mean_put, "drain_ms": mean_drain,
                   "put_GBps": sb["put"] / (mean_put * 1e-3) / 1e9,
                   "drain_GBps": sb["get_hbm"] / (mean_drain * 1e-3) / 1e9,
                   "drain_delivered_GBps": sb["get_delivered"] / (mean_drain * 1e-3) / 1e9,
                   "step_GBps": (sb["put"] + sb["get_hbm"]) / (ms_per_step * 1e-3) / 1e9,
                   "step_frac_of_measured_copy": (sb["put"] + sb["get_hbm"]) / (ms_per_step * 1e-3) / 1e9 / peak},
        "gpu_launches": launches, "gpu_launches_per_step": launches // steps, "clocks": clocks,
    }
    if not brief:
        # per-kernel pass: event pairs around every launch of the two copy kernels
        step.dock.kernel_timing(True)
        ksteps = min(args.steps, 5)
        for _ in range(ksteps):
            step.timed_step()
        n_sc, ms_sc = step.dock.kernel_timing_read(0)
        n_ga, ms_ga = step.dock.kernel_timing_read(1)
        step.dock.kernel_timing(False)
        kern = {"put_scatter": kernel_record(ms_sc, n_sc, ksteps, sb["put_ragged"], sb["put_ragged"], peak),
                "get_gather": kernel_record(ms_ga, n_ga, ksteps, sb["get_hbm"], sb["get_delivered"], peak)}
        dom = "get_gather" if ms_ga >= ms_sc else "put_scatter"
        k = kern[dom]
        traffic = (None if (args.fused or args.padded or warm_l2 or sigma is not None or args.api != "many")
                   else captured_traffic(cid, dom, k["bytes_per_launch"]))
        rec["kernels"] = kern
        rec["roofline"] = {
            # numerator: the bytes that must cross HBM in one launch (every stored row that is taken
            # read once, every delivered byte written once); a launch that serves several consumers
            # reads a row once from HBM and again from L2, which `delivered` counts and this does not
            "bound": "hbm" if k["frac_of_measured_copy"] >= 0.5 else "latency",
            "kernel": dom, "achieved": k["GBps"], "peak": peak, "unit": "GB/s", "frac": k["frac_of_measured_copy"],
            "frac_of_nominal_8TBps": k["frac_of_nominal_8TBps"],
            "traffic": traffic[0] if traffic else None,
            "traffic_source": (f"{traffic[1]} ({traffic[2]}); not observed by this run" if traffic else None),
            "peak_kind": peak_kind, "bytes_per_launch": k["bytes_per_launch"], "avg_launch_ms": k["avg_ms"],
            "delivered_GBps": k["delivered_GBps"],
            "numerator": "bytes that must cross HBM per launch: stored rows read once + delivered bytes written",
        }
        if warm_l2:
            rec["roofline"]["bound"] = "l2-assisted" if k["frac_of_measured_copy"] > 1.0 else rec["roofline"]["bound"]
    e2e = None
    if with_e2e and not brief and not args.no_e2e and not args.padded:
        e2e_s, d2h, copies = step.run_e2e(min(args.steps, 5), 1)
        e2e_s, = max_over_ranks(dist, [e2e_s], step.dev)
        e2e = {"value": whole_job_rate(world, n_dispatch, e2e_s), "unit": "samples/s", "ms_per_step": e2e_s * 1e3,
               "h2d_bytes_per_step": getattr(step, "e2e_h2d_bytes", None) or step.h2d_bytes, "d2h_bytes_per_step": d2h}
        e2e.update(copies)
    rec["e2e"] = e2e
    step.close()
    del step
    cpu = None
    if with_cpu and not brief and rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import td_oracle
        td_oracle.build()
        rate, steps_o, el = time_oracle(w, args.cpu_seconds)
        cpu = {"value": rate, "unit": "samples/s", "cores": 1, "kind": "oracle",
               "sample": f"{steps_o} whole step(s) of the same workload in {el:.1f} s"}
        if not args.no_cpu_all_cores:
            rate_all, procs, el_all = time_oracle_all_cores(cid, sigma, args.cpu_seconds)
            cpu["all_cores"] = {"value": rate_all, "unit": "samples/s", "cores": procs, "kind": "oracle",
                                "sample": f"{procs} processes, one dock each over the same workload, whole steps "
                                          f"for {el_all:.1f} s; host has {os.cpu_count()} logical cores"}
    rec["cpu_baseline"] = cpu
    return rec


# --------------------------------------------------------------------------- the out-of-order stress
def run_concurrent(args, cid: int, rank: int, local_rank: int, sigma=None):
    """One producer thread putting the shape's columns in seeded random chunks of 1-64 samples on
    its own stream while four consumer threads poll td_get on theirs until each has been served
    every sample.  Wall-clock time (the polling loop is the host's); exactly-once dispatch is
    checked from the served marks and counters before anything is reported."""
    import torch
    from paper_2507_19017_b200 import binding as td
    from paper_2507_19017_b200 import workloads as wl
    w = make_workload(cid, rank, sigma, "interleaved")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dock = td.Dock(w.G, w.N, w.S, w.column_tuples(), w.consumer_tuples(),
                   w.shard_capacity(wl.PROMPT), w.shard_capacity(wl.RESPONSE), w.column_index("reward"), 1e-6, local_rank)

    def to_dev(a):
        t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else np.ascontiguousarray(a))
        return (t.view(torch.bfloat16) if a.dtype == np.uint16 else t).to(dev)

    # every put's arrays are resident before the clock starts: per column one index array, one cu
    # array and one data array holding the chunks back to back
    puts = [op for op in w.ops if op.kind == "put"]
    per_col = {}
    for op in puts:
        per_col.setdefault(op.column, []).append(op)
    calls = {}
    for col, ops in per_col.items():
        idx_parts, cu_parts, data_parts = [], [], []
        for op in ops:
            cu, data = w.pack(col, op.indices)
            idx_parts.append(np.ascontiguousarray(op.indices, np.int32)); cu_parts.append(cu); data_parts.append(data)
        d_idx = to_dev(np.concatenate(idx_parts))
        d_cu = to_dev(np.concatenate(cu_parts)) if cu_parts[0] is not None else None
        d_data = to_dev(np.concatenate(data_parts))
        i0 = c0 = e0 = 0
        for op, ip, cp, dp in zip(ops, idx_parts, cu_parts, data_parts):
            # a slice of length zero has no address of its own: a put of empty rows still gets a valid pointer
            data_view = d_data[e0:e0 + len(dp)] if len(dp) else d_data[:0]
            calls[id(op)] = (col, d_idx[i0:i0 + len(ip)], d_cu[c0:c0 + len(cp)] if d_cu is not None else None, data_view)
            i0 += len(ip); e0 += len(dp)
            if cp is not None:
                c0 += len(cp)
    order = [calls[id(op)] for op in puts]
    lp = np.sort(w.len_prompt)[::-1]
    lr = np.sort(w.len_response)[::-1]
    m = w.micro_batch
    n_c = len(w.consumers)
    bufs = [td.GetBuffers(dock, c, m, td.PACKED, prompt_tokens_cap=int(lp[:m].sum(dtype=np.int64)),
                          response_tokens_cap=int(lr[:m].sum(dtype=np.int64))) for c in range(n_c)]
    # result blocks in pinned host memory: the polling thread reads the count without another copy
    results = [torch.zeros(32, dtype=torch.uint8).pin_memory() for _ in range(n_c)]
    for b, r in zip(bufs, results):
        b.struct.result = r.data_ptr()
    stats = [{"gets": 0, "empty": 0, "samples": 0, "tokens": 0} for _ in range(n_c)]
    errors = []
    start = threading.Barrier(n_c + 2)
    done_putting = threading.Event()

    def producer():
        try:
            s = torch.cuda.Stream(device=dev)
            start.wait()
            for col, idx, cu, data in order:
                dock.put(col, idx, cu, data, stream=s)
            s.synchronize()
        except Exception as e:          # pragma: no cover
            errors.append(e)
        finally:
            done_putting.set()

    def consumer(c):
        try:
            s = torch.cuda.Stream(device=dev)
            res = td.TdResult.from_address(results[c].data_ptr())
            st = stats[c]
            start.wait()
            deadline = time.time() + 300
            idle = 0
            while st["samples"] < w.n:
                dock.get(bufs[c], stream=s)
                s.synchronize()
                st["gets"] += 1
                if res.status:
                    raise RuntimeError(f"consumer {c}: get reported status {res.status:#x}")
                if res.n_samples:
                    st["samples"] += res.n_samples
                    st["tokens"] += res.prompt_tokens + res.response_tokens
                    idle = 0
                else:
                    st["empty"] += 1
                    idle += done_putting.is_set()
                    if idle > 5000 or time.time() > deadline:
                        raise RuntimeError(f"consumer {c} cannot drain the dock ({st})")
        except Exception as e:
            errors.append(e)

    threads = [threading.Thread(target=producer)] + [threading.Thread(target=consumer, args=(c,)) for c in range(n_c)]
    for t in threads:
        t.start()
    start.wait()
    t0 = time.perf_counter()
    for t in threads:
        t.join(timeout=330)
    wall = time.perf_counter() - t0
    if errors or any(t.is_alive() for t in threads):
        raise errors[0] if errors else RuntimeError("a thread of the concurrent scenario did not finish")
    torch.cuda.synchronize()
    # exactly once: every consumer was served n samples, its served marks cover every sample once
    # (a group served twice would count twice in got_samples), every group is claimed
    st = dock.status()
    rep = dock.validate()
    for c in range(n_c):
        ok = (stats[c]["samples"] == w.n and st.got_samples[c] == w.n and rep.served[c] == w.n)
        if not ok or rep.violations or st.error_word:
            raise RuntimeError(f"exactly-once check failed for consumer {c}: thread saw {stats[c]['samples']}, "
                               f"counter {st.got_samples[c]}, served marks {rep.served[c]}, "
                               f"violations {rep.violations:#x}, error word {st.error_word:#x}")
    launches = dock.launch_count()
    rec = {"scenario": "one producer stream (seeded random chunks of 1-64 samples per column), four consumer host "
                       "threads polling td_get on their own streams",
           "workload": f"configs[{cid - 1}] {w.name}", "samples": w.n, "tokens": w.tokens_total(),
           "wall_ms": wall * 1e3, "value": n_c * w.n / wall, "unit": "samples/s",
           "tokens_per_s": sum(s["tokens"] for s in stats) / wall,
           "put_calls": len(order), "gets_issued": sum(s["gets"] for s in stats),
           "empty_gets": sum(s["empty"] for s in stats), "partial_or_full_gets": sum(s["gets"] - s["empty"] for s in stats),
           "n_claim_conflicts": int(st.n_claim_conflicts), "gpu_launches": int(launches),
           "exactly_once": "verified: per consumer the thread's count, got_samples and the served marks all equal n; "
                           "no validate violation, error word 0",
           "timing": "wall clock from the common start of the five threads to the last join"}
    dock.close()
    del dock, bufs, order, calls
    torch.cuda.empty_cache()
    return rec


# --------------------------------------------------------------------------- main
def reference_arm(args, rank: int):
    """The oracle as it stands on the headline shape: `warmup` untimed and `steps` timed whole
    steps on one host core (cut short when they would take minutes)."""
    if rank != 0:
        return
    from oracle import td_oracle
    td_oracle.build()
    cid = args.config or HEADLINE_CONFIG
    w = make_workload(cid, 0, args.sigma, "bulk")
    config = config_dict(w, cid, args.sigma, args.warm_l2)
    rate, steps, el = time_oracle(w, max(args.cpu_seconds, 0.1), steps=max(args.steps, 1), warmup=args.warmup)
    line = {"metric": METRIC, "value": rate, "unit": "samples/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * el / steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
            "data": "synthetic", "impl": "reference", "config": config,
            "cpu_baseline": {"value": rate, "unit": "samples/s", "cores": 1, "kind": "oracle",
                             "sample": f"{steps} whole step(s) of the workload in {el:.1f} s"},
            "e2e": {"value": rate, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        reference_arm(args, rank)
        return

    import torch
    from paper_2507_19017_b200 import build
    build.build()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback")
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def finish():
        if dist is not None:
            dist.destroy_process_group()

    if args.scenario == "scan":
        if rank == 0:
            run_scan(args, local_rank)
        return finish()
    if args.scenario == "fixed-cost":
        if rank == 0:
            run_fixed_cost(args, local_rank)
        return finish()
    if args.scenario == "cascade":
        from paper_2507_19017_b200 import workloads as wl
        cid = args.config or 2
        w = make_workload(cid, rank, args.sigma, "cascade_batched" if args.api == "many" else "cascade")
        run_cascade(args, w, local_rank, world, dist, config_dict(w, cid, args.sigma, args.warm_l2))
        return finish()
    if args.scenario == "concurrent":
        rec = run_concurrent(args, args.config or 4, rank, local_rank, args.sigma)
        if rank == 0:
            print(json.dumps(dict(rec, metric=METRIC, n_gpus=world, higher_is_better=True, data="synthetic")))
        return finish()

    configs = [args.config] if args.config else list(DEFAULT_CONFIGS)
    sampler = make_sampler(torch, local_rank)
    sampler.start()
    records = []
    for cid in configs:
        rec = measure_dispatch(args, cid, rank, local_rank, world, dist, sampler, sigma=args.sigma, warm_l2=args.warm_l2)
        if not args.no_variants and not args.warm_l2 and args.sigma is None and not (args.fused or args.padded):
            variants = {"warm_l2": measure_dispatch(args, cid, rank, local_rank, world, dist, sampler, warm_l2=True, brief=True)}
            if cid == configs[0]:
                variants["response_sigma_0.75"] = measure_dispatch(args, cid, rank, local_rank, world, dist, sampler,
                                                                   sigma=0.75, brief=True)
            rec["variants"] = {k: {kk: v[kk] for kk in ("config", "value", "ms_per_step", "ms_per_step_median",
                                                        "ms_per_step_min", "tokens_per_s", "phases")}
                               for k, v in variants.items()}
        if cid == 4 and not args.config and not (args.fused or args.padded) and world == 1:
            rec["concurrent"] = run_concurrent(args, 4, rank, local_rank, args.sigma)
        records.append(rec)
    sampler.stop()
    if rank != 0:
        return finish()
    head = records[0]
    line = {
        "metric": METRIC, "value": head["value"], "unit": "samples/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic", "config": head["config"],
    }
    for k in ("api", "ms_per_step_median", "ms_per_step_min", "spread", "tokens_per_s", "phases", "kernels", "roofline",
              "cpu_baseline", "e2e", "gpu_launches", "gpu_launches_per_step", "clocks", "variants"):
        if k in head:
            line[k] = head[k]
    line["per_config"] = sorted(records, key=lambda r: r["config"]["workload"])
    print(json.dumps(line))
    finish()


if __name__ == "__main__":
    main()
