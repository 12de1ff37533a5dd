#!/usr/bin/env python
"""Benchmark of the transfer dock's put/get dispatch.

One step = one pass of the whole hot path over one synthetic GRPO batch: reset the dock, put
every column of every sample, then drain it for all consumers in micro-batches.  The headline
value is samples dispatched to consumers per second of (put phase + drain phase), with inputs
resident in HBM.  The L2 is flushed (a 256 MiB write, untimed) before each phase.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl reference]
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
# DRAM bytes (read + write) of one launch, from the ncu capture summarised under profiles/ for
# the kernels as built; (config, kernel) pairs without a capture report null.
NCU_TRAFFIC = {(2, "get_gather"): 79_587_584, (2, "put_scatter"): 44_971_776,
               (3, "get_gather"): 1_147_116_032, (3, "put_scatter"): 732_750_848}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2, help="workload shape 1..5 (default 2: Qwen2.5-7B-shaped)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--api", default="many", choices=["many", "single"],
                    help="many: one td_put_many and one td_get_many per step; single: one td_put per "
                         "column and one td_get per micro-batch")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="CPU-oracle time budget")
    ap.add_argument("--fused", action="store_true",
                    help="the actor update's gets also ask for the fused prompt+response id stream and "
                         "its per-token advantage twin")
    ap.add_argument("--padded", action="store_true",
                    help="gets write right-padded rows (row i at i * width, the column's pad bits behind it) "
                         "instead of packed ones; widths are the workload's maximum lengths")
    ap.add_argument("--graph", action="store_true",
                    help="cascade only: capture the step's calls into one CUDA graph once and time its replay "
                         "(nothing in the step needs the host, batch sizes are read on the device)")
    ap.add_argument("--scenario", default="dispatch", choices=["dispatch", "cascade", "scan"],
                    help="dispatch: put everything, then drain (the headline); cascade: generation puts in "
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

    def stop(self, t_begin: float, t_end: float):
        """Summary of the samples taken inside [t_begin, t_end] (the timed region); when the
        region was too short to catch three, of everything sampled since start (warm-up and
        timed region, both under the same load)."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
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

        inside = [(t, ln) for t, ln in self.lines if t_begin <= t <= t_end + 0.03]
        window = "timed region"
        sm, mx, reasons = summarise(inside)
        if len(sm) < 3:
            window = "warm-up and timed region"
            sm, mx, reasons = summarise(self.lines)
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

    def stop(self, t_begin: float, t_end: float, t_soak_end: float = 0.0):
        self.stop_flag.set()
        if self.thread:
            self.thread.join(timeout=2)
        inside = [s for s in self.samples if t_begin <= s[0] <= t_end]
        window = "timed region"
        if len(inside) < 3 and t_soak_end > t_end:
            inside = [s for s in self.samples if t_begin <= s[0] <= t_soak_end]
            window = "timed region and the same steps repeated right after it (the region is a few ms)"
        if len(inside) < 3:
            inside, window = self.samples, "warm-up and timed region"
        reasons = set()
        for _t, _mhz, bits in inside:
            for bit, name in self.REASONS.items():
                if bits & bit:
                    reasons.add(name)
        sm = [s[1] for s in inside]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": self.max_mhz,
                "samples": len(sm), "window": window, "source": "nvml", "reasons": sorted(reasons)}


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
def algorithmic_bytes(w):
    """Bytes the method must move per step: every put row read and written once, every served
    row read and written once, element size times true length (no padding)."""
    from paper_2507_19017_b200 import workloads as wl
    put = 0
    for spec in w.columns:
        put += 2 * w.data[spec.name].nbytes
    put_ragged = sum(2 * w.data[s.name].nbytes for s in w.columns if s.cls != wl.SCALAR)
    get = 0
    for k in w.consumers:
        for name in k.out:
            get += 2 * w.data[name].nbytes
    return put, put_ragged, get


class GpuStep:
    """Device-resident inputs and per-get output buffers of one step, and the step itself."""

    def __init__(self, w, device_index: int, api: str = "many", fused: bool = False, padded: bool = False):
        import torch
        self.api = api
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
        self.flush_buf.zero_()

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
        td, torch = self.td, self.torch
        needs = [self.dock.put_host_stage_bytes(c, i.numel(), d.numel()) for c, i, _cu, d in self.host_puts]
        if self.api == "many":
            self.stage = [torch.empty(sum(needs), dtype=torch.uint8, device=self.dev)]
        else:
            self.stage = [torch.empty(max(needs), dtype=torch.uint8, device=self.dev) for _ in range(2)]
        self.host_gets = [td.HostGetBuffers(b) for b in self.gets]
        self.host_put_arr = self.dock.put_items(self.host_puts)       # marshalled once, like a caller would
        self.host_out_arr = self.dock.host_outs(self.host_gets)
        self.meta_stage = (torch.empty(self.dock.get_many_host_stage_bytes(self.plan), dtype=torch.uint8, device=self.dev)
                           if self.api == "many" else None)

    def e2e_step(self):
        torch = self.torch
        self.dock.reset()
        if self.api == "many":          # one call in, one call out: two synchronisations per step
            self.dock.put_many_host(self.host_put_arr, self.stage[0])
            self.dock.get_many_host(self.plan, self.host_out_arr, self.meta_stage)
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
        return el, sum(h.bytes_valid(self.dock) for h in self.host_gets)      # counted from what the last step copied


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
    graph, step.graph = step.graph, None                    # the per-kernel pass below runs eagerly
    # algorithmic bytes: every stored row read and written once, every served row read and written once
    _put, _ragged, get_bytes = algorithmic_bytes(w)
    put_bytes = sum(2 * w.data[s.name].nbytes for s in w.columns)
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
        "roofline": {"bound": "hbm", "kernel": dom, "achieved": kern[dom]["GBps"], "peak": peak, "unit": "GB/s",
                     "frac": kern[dom]["GBps"] / peak, "traffic": None, "peak_kind": peak_kind,
                     "bytes_per_launch": kern[dom]["bytes_per_launch"], "avg_launch_ms": kern[dom]["avg_ms"],
                     "note": "average over many small launches: this scenario is bound by launch latency"},
        "cpu_baseline": None, "e2e": None,
        "gpu_launches": launches, "gpu_launches_per_step": launches // args.steps, "clocks": clocks,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- CPU oracle
def time_oracle(w, budget_s: float):
    """The oracle as it stands, one thread, whole steps of the same workload until the time
    budget is used (at least one step).  Returns (samples/s, steps, seconds)."""
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
    gets = []
    for op in w.ops:
        if op.kind == "get":
            m = op.max_samples
            caps = {}
            for c, (dt, cls, _p) in enumerate(d.columns):
                caps[c] = m if cls == 0 else int((lp if cls == 1 else lr)[:m].sum(dtype=np.int64))
            gets.append(d.prepare_get(op.consumer, m, caps))
    steps, samples = 0, 0
    t0 = time.perf_counter()
    while True:
        d.reset()
        for col, idx, cu, data in puts:
            d.put_raw(col, idx, cu, data)
        for g in gets:
            samples += d.get_prepared(g)
        steps += 1
        el = time.perf_counter() - t0
        if el >= budget_s:
            break
    d.close()
    return samples / el, steps, el


# --------------------------------------------------------------------------- main
def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2507_19017_b200 import workloads as wl
    schedule = "bulk" if args.scenario == "dispatch" else ("cascade_batched" if args.api == "many" else "cascade")
    w = wl.make_config(args.config, seed=wl.BASE_SEED + args.config + 1000 * rank, schedule=schedule)
    config = {"workload": f"configs[{args.config - 1}] {w.name}", "G": w.G, "N": w.N, "S": w.S,
              "samples": w.n, "tokens": w.tokens_total(), "micro_batch": w.micro_batch,
              "consumers": len(w.consumers), "schedule": "one put per column, then round-robin gets",
              "l2": "flushed before each phase (256 MiB write)", "response_sigma": wl.SIGMA_HEADLINE}
    n_dispatch = w.n * len(w.consumers)

    if args.impl == "reference":
        if rank != 0:
            return
        from oracle import td_oracle
        td_oracle.build()
        steps_s = []
        for _ in range(args.warmup):
            pass          # the oracle needs no warm-up beyond its first pass, which is timed too
        rate, steps, el = time_oracle(w, max(args.cpu_seconds, 1.0))
        line = {"metric": METRIC, "value": rate, "unit": "samples/s", "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * el / steps,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
                "data": "synthetic", "impl": "reference", "config": config,
                "cpu_baseline": {"value": rate, "unit": "samples/s", "cores": 1, "kind": "oracle",
                                 "sample": f"{steps} whole step(s) of the workload in {el:.1f} s"},
                "e2e": {"value": rate, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
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

    if args.scenario == "scan":
        if rank == 0:
            run_scan(args, local_rank)
        if dist is not None:
            dist.destroy_process_group()
        return
    if args.scenario == "cascade":
        run_cascade(args, w, local_rank, world, dist, config)
        if dist is not None:
            dist.destroy_process_group()
        return

    step = GpuStep(w, local_rank, args.api, args.fused, args.padded)
    if args.padded:
        config["output"] = f"right-padded rows, widths {w.pad_prompt_to} / {w.pad_response_to}"
    if args.fused:
        config["fused_stream"] = "actor-update gets also write the prompt+response id stream and its advantage twin"
    config["api"] = ("td_put_many + td_get_many (one call each per step)" if args.api == "many"
                     else "td_put per column + td_get per micro-batch")
    peak, peak_kind = load_peaks()
    put_bytes, put_ragged_bytes, get_bytes = algorithmic_bytes(w)
    if args.padded:      # the pad writes are part of what this mode must move
        from paper_2507_19017_b200 import workloads as wl_
        for k in w.consumers:
            for name in k.out:
                spec = w.columns[w.column_index(name)]
                if spec.cls != wl_.SCALAR:
                    width = w.pad_prompt_to if spec.cls == wl_.PROMPT else w.pad_response_to
                    get_bytes += (w.n * width * w.data[name].itemsize) - w.data[name].nbytes

    if args.fused:       # the stream: both id columns read and written once more; the twin: one float written per token
        get_bytes += 2 * (w.data["prompt_ids"].nbytes + w.data["response_ids"].nbytes) + 4 * w.tokens_total()

    sampler = make_sampler(torch, local_rank)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step.timed_step()
    served_s, served_t = step.served()
    assert served_s == n_dispatch, f"drain served {served_s} of {n_dispatch} samples"

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    barrier()
    t_begin = time.time()
    torch.cuda.cudart().cudaProfilerStart()        # lets a profiler capture the timed region only
    launches0 = step.dock.launch_count()
    put_ms, drain_ms = [], []
    for _ in range(args.steps):
        a, b = step.timed_step()
        put_ms.append(a); drain_ms.append(b)
    barrier()
    torch.cuda.cudart().cudaProfilerStop()
    t_end = time.time()
    launches = step.dock.launch_count() - launches0
    # A timed region of a few milliseconds holds too few clock samples: the same steps go on,
    # untimed, until the sampler has seen the device under this load for a while.
    t_soak_end = t_end
    if isinstance(sampler, NvmlSampler) and sampler.count_inside(t_begin, t_end) < 3:
        while time.time() - t_end < 0.25 and sampler.count_inside(t_begin, time.time()) < 8:
            step.timed_step()
        t_soak_end = time.time()
    clocks = sampler.stop(t_begin, t_end, t_soak_end) if isinstance(sampler, NvmlSampler) else sampler.stop(t_begin, t_end)

    mean_put, mean_drain = sum(put_ms) / len(put_ms), sum(drain_ms) / len(drain_ms)
    ms_per_step = mean_put + mean_drain
    ms_per_step, mean_put, mean_drain = max_over_ranks(dist, [ms_per_step, mean_put, mean_drain], step.dev)
    value = whole_job_rate(world, n_dispatch, ms_per_step * 1e-3)

    # per-kernel pass: event pairs around every launch of the two copy kernels
    step.dock.kernel_timing(True)
    ksteps = min(args.steps, 5)
    for _ in range(ksteps):
        step.timed_step()
    n_sc, ms_sc = step.dock.kernel_timing_read(0)
    n_ga, ms_ga = step.dock.kernel_timing_read(1)
    step.dock.kernel_timing(False)
    kern = {
        "put_scatter": {"launches_per_step": n_sc // ksteps, "avg_ms": ms_sc / max(n_sc, 1),
                        "bytes_per_launch": put_ragged_bytes / max(n_sc // ksteps, 1)},
        "get_gather": {"launches_per_step": n_ga // ksteps, "avg_ms": ms_ga / max(n_ga, 1),
                       "bytes_per_launch": get_bytes / max(n_ga // ksteps, 1)},
    }
    for k in kern.values():
        k["GBps"] = k["bytes_per_launch"] / (k["avg_ms"] * 1e-3) / 1e9 if k["avg_ms"] > 0 else 0.0
    dom = "get_gather" if ms_ga >= ms_sc else "put_scatter"
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kern[dom]["GBps"], "peak": peak, "unit": "GB/s",
                "frac": kern[dom]["GBps"] / peak, "traffic": None if (args.fused or args.padded) else NCU_TRAFFIC.get((args.config, dom)),
                "peak_kind": peak_kind,
                "bytes_per_launch": kern[dom]["bytes_per_launch"], "avg_launch_ms": kern[dom]["avg_ms"]}

    e2e = None
    if not args.no_e2e and not args.padded:
        e2e_s, d2h = step.run_e2e(min(args.steps, 5), 1)
        e2e_s, = max_over_ranks(dist, [e2e_s], step.dev)
        e2e = {"value": whole_job_rate(world, n_dispatch, e2e_s), "unit": "samples/s", "ms_per_step": e2e_s * 1e3,
               "h2d_bytes_per_step": step.h2d_bytes, "d2h_bytes_per_step": d2h}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import td_oracle
        td_oracle.build()
        rate, steps_o, el = time_oracle(w, args.cpu_seconds)
        cpu = {"value": rate, "unit": "samples/s", "cores": 1, "kind": "oracle",
               "sample": f"{steps_o} whole step(s) of the same workload in {el:.1f} s"}

    line = {
        "metric": METRIC, "value": value, "unit": "samples/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic", "config": config,
        "tokens_per_s": world * served_t / (ms_per_step * 1e-3),
        "phases": {"put_ms": mean_put, "drain_ms": mean_drain,
                   "put_GBps": put_bytes / (mean_put * 1e-3) / 1e9,
                   "drain_GBps": get_bytes / (mean_drain * 1e-3) / 1e9,
                   "step_GBps": (put_bytes + get_bytes) / (ms_per_step * 1e-3) / 1e9},
        "kernels": kern, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
        "gpu_launches": launches, "gpu_launches_per_step": launches // args.steps, "clocks": clocks,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
