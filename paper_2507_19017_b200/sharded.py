"""One transfer dock sharded over several GPUs, one process per GPU.

"Distributed Transfer Dock Strategy" splits the buffer along the global batch into S
warehouses and keeps the controllers' metadata consistent by a small broadcast (the
8(C+1)M / S term of Eq. 4).  Here warehouse j lives on rank j mod P, inside that rank's own
dock (the CUDA library; its kernels do every put, select, claim, gather and advantage of the
rows that rank owns).  What this module adds is the part between the ranks:

  put    a collective: every rank hands in the rows it produced, whatever their owners; rows
         travel to the rank that owns their warehouse (one all-to-all of indices, lengths and
         payload) and are put into its local dock.
  sync   the metadata broadcast: an all-gather of the local status words and claim bits gives
         every rank the same replica of the readiness of all samples.
  get    a collective on behalf of one worker state, whose batch is delivered to its home rank
         (consumer c lives on rank c mod P unless told otherwise).  Every rank derives the same
         selection from its replica - the lowest ready, unclaimed groups - which fixes how many
         groups each rank contributes; because warehouses hold contiguous blocks of prompts,
         the part of a lowest-first selection that falls on one rank is again the lowest ready
         groups of that rank, so each owner simply asks its local dock for that many samples.
         The owners' packed rows then travel to the home rank, which lays them out in global
         group order and rebuilds cu_seqlens from the lengths.

No data-path collective exists inside a rank's dock, and no kernel, this library's or anyone's,
is handed another GPU's memory: the exchange is torch.distributed (NCCL on GPUs, gloo in the CPU
tests) into local buffers.  With one rank every exchange
degenerates to a local copy and the results are those of the plain dock.

The local dock is reached through a small adapter (`CudaLocal` below; the tests plug a CPU
stand-in into the same seam), so that the routing, the replica and the assembly can be checked
without a GPU.  Measured on hardware: not yet (one GPU per run so far).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import torch


# --------------------------------------------------------------------------- index arithmetic
class ShardMap:
    """Which rank owns which warehouse, and the local numbering on that rank.

    Warehouse (shard) j holds the prompts [j * gps, (j + 1) * gps), gps = G / S; it lives on rank
    j mod P as that rank's local shard j div P.  Local group / sample numbers follow from the
    local shard number the same way global ones follow from the global shard number."""

    def __init__(self, G: int, N: int, S: int, P: int):
        if G % S or P < 1 or S < P:
            raise ValueError("need S | G and at least one warehouse per rank")
        self.G, self.N, self.S, self.P = G, N, S, P
        self.gps = G // S
        self.n = G * N

    def shards_of(self, rank: int) -> List[int]:
        return list(range(rank, self.S, self.P))

    def local_shape(self, rank: int):
        """(G_local, S_local) of the dock rank `rank` holds."""
        s_local = len(self.shards_of(rank))
        return s_local * self.gps, s_local

    def owner_of_group(self, g: torch.Tensor) -> torch.Tensor:
        return (g // self.gps) % self.P

    def local_group(self, g: torch.Tensor) -> torch.Tensor:
        shard = g // self.gps
        return (shard // self.P) * self.gps + g % self.gps

    def global_group(self, rank: int, lg: torch.Tensor) -> torch.Tensor:
        shard = (lg // self.gps) * self.P + rank
        return shard * self.gps + lg % self.gps

    def local_sample(self, s: torch.Tensor) -> torch.Tensor:
        return self.local_group(s // self.N) * self.N + s % self.N

    def global_sample(self, rank: int, ls: torch.Tensor) -> torch.Tensor:
        return self.global_group(rank, ls // self.N) * self.N + ls % self.N

    def global_samples_of(self, rank: int) -> torch.Tensor:
        """Global sample numbers of rank `rank`'s local samples, in local order."""
        g_local, _ = self.local_shape(rank)
        return self.global_sample(rank, torch.arange(g_local * self.N, dtype=torch.int64))


# --------------------------------------------------------------------------- communication
class Comm:
    """The three exchanges the sharded dock needs, over torch.distributed or, alone, over nothing."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist = dist if (dist.is_available() and dist.is_initialized()) else None
        self.group = group
        self.rank = self.dist.get_rank(group) if self.dist else 0
        self.world = self.dist.get_world_size(group) if self.dist else 1

    def all_to_all(self, send: torch.Tensor, send_counts: Sequence[int], recv_counts: Sequence[int]) -> torch.Tensor:
        """1-D tensors; send_counts[r] leading-to-trailing elements go to rank r."""
        out = torch.empty(int(sum(recv_counts)), dtype=send.dtype, device=send.device)
        if self.world == 1:
            out.copy_(send)
            return out
        self.dist.all_to_all_single(out, send.contiguous(), output_split_sizes=[int(c) for c in recv_counts],
                                    input_split_sizes=[int(c) for c in send_counts], group=self.group)
        return out

    def exchange_counts(self, counts: Sequence[int], device) -> List[int]:
        """counts[r] = what this rank sends to r; returns what it receives from each rank."""
        if self.world == 1:
            return [int(counts[0])]
        send = torch.tensor([int(c) for c in counts], dtype=torch.int64, device=device)
        recv = torch.empty_like(send)
        self.dist.all_to_all_single(recv, send, group=self.group)
        return [int(c) for c in recv.tolist()]

    def all_gather_padded(self, x: torch.Tensor, sizes: Sequence[int]) -> List[torch.Tensor]:
        """x has sizes[rank] elements; returns every rank's x."""
        if self.world == 1:
            return [x]
        width = max(int(s) for s in sizes)
        mine = torch.zeros(width, dtype=x.dtype, device=x.device)
        mine[:x.numel()] = x
        parts = [torch.empty(width, dtype=x.dtype, device=x.device) for _ in range(self.world)]
        self.dist.all_gather(parts, mine, group=self.group)
        return [p[:int(s)] for p, s in zip(parts, sizes)]


# --------------------------------------------------------------------------- batches
@dataclass
class LocalBatch:
    """What a rank's own dock served: samples in local numbering, rows packed."""
    n_samples: int
    indices: torch.Tensor                      # int32 [n] local sample numbers, ascending
    cu_prompt: torch.Tensor                    # int32 [n + 1]
    cu_response: torch.Tensor                  # int32 [n + 1]
    columns: Dict[int, torch.Tensor] = field(default_factory=dict)     # packed (scalar columns: [n])
    advantages: Optional[torch.Tensor] = None  # float32 [n]


@dataclass
class ShardedBatch:
    """A batch as the home rank of a worker state receives it: global sample numbers, rows packed
    in global group order."""
    n_samples: int
    n_groups: int
    indices: torch.Tensor
    cu_prompt: torch.Tensor
    cu_response: torch.Tensor
    cu_seq: torch.Tensor
    columns: Dict[int, torch.Tensor]
    advantages: Optional[torch.Tensor]
    prompt_tokens: int = 0
    response_tokens: int = 0


def _as_bytes(t: torch.Tensor) -> torch.Tensor:
    return t.contiguous().view(torch.uint8).reshape(-1)


# --------------------------------------------------------------------------- the sharded dock
class ShardedDock:
    """columns: (dtype tag, class tag, pad_bits) as for binding.Dock; consumers: (need_mask,
    out_mask, advantage).  `local` is this rank's own dock behind the adapter interface:
        put(column, indices int32, cu int32 or None, data)      get(consumer, max_samples) -> LocalBatch
        status_words() -> int32 [n_local]                        claim_bits(consumer) -> bool [G_local]
        reset()                                                  device"""

    ELEM = {"i32": (torch.int32, 4), "f32": (torch.float32, 4), "bf16": (torch.bfloat16, 2)}

    def __init__(self, smap: ShardMap, local, comm: Comm, columns: Sequence, consumers: Sequence):
        self.map, self.local, self.comm = smap, local, comm
        self.rank, self.P = comm.rank, comm.world
        if self.P != smap.P:
            raise ValueError("the shard map was made for another number of ranks")
        self.columns = list(columns)
        self.consumers = [(int(a), int(b), bool(f)) for a, b, f in consumers]
        self.device = local.device
        self._n_local = [smap.local_shape(r)[0] * smap.N for r in range(self.P)]
        self._g_local = [smap.local_shape(r)[0] for r in range(self.P)]
        self._glob_samples = [smap.global_samples_of(r).to(self.device) for r in range(self.P)]
        self._glob_groups = [smap.global_group(r, torch.arange(self._g_local[r], dtype=torch.int64)).to(self.device)
                             for r in range(self.P)]
        self.status = torch.zeros(smap.n, dtype=torch.int32, device=self.device)           # replica
        self.claimed = torch.zeros(len(self.consumers), smap.G, dtype=torch.bool, device=self.device)

    def home_of(self, consumer: int) -> int:
        return consumer % self.P

    # -- workflow steps 2 and 3, producer side ------------------------------------------------
    def put(self, column: int, indices: torch.Tensor, cu: Optional[torch.Tensor], data: torch.Tensor) -> None:
        """Collective.  indices: global sample numbers (int32, any owners, any order); cu int32
        [k + 1] or None for a scalar column; data: rows back to back.  A rank with nothing to put
        passes empty tensors."""
        m, dev = self.map, self.device
        dtype, esz = self.ELEM[self.columns[column][0]]
        idx = indices.to(dev).to(torch.int64).reshape(-1)
        k = idx.numel()
        ragged = self.columns[column][1] != "scalar"
        if ragged:
            cu64 = cu.to(dev).to(torch.int64)
            lens = cu64[1:] - cu64[:-1]
            starts = cu64[:-1]
            # rows travel as (length, elements): an array that goes down somewhere cannot be sent on
            if k and (bool((lens < 0).any()) or int(cu64[0]) < 0 or int(cu64[-1]) > data.numel()):
                raise ValueError("cu must be non-decreasing and lie inside data")
        else:
            lens = torch.ones(k, dtype=torch.int64, device=dev)
            starts = torch.arange(k, dtype=torch.int64, device=dev)
        valid = (idx >= 0) & (idx < m.n)
        safe = torch.where(valid, idx, torch.zeros_like(idx))
        dest = torch.where(valid, m.owner_of_group(safe // m.N), torch.zeros_like(idx))
        local_idx = torch.where(valid, m.local_sample(safe), torch.full_like(idx, -1))     # an index out of range stays one
        order = torch.sort(dest, stable=True).indices                                       # rows by owner, call order kept
        send_rows = torch.bincount(dest, minlength=self.P).tolist() if k else [0] * self.P
        lens_s, starts_s = lens[order], starts[order]
        # the rows' elements, owner by owner (a ragged gather)
        take = lens_s
        row_of = torch.repeat_interleave(torch.arange(k, device=dev), take)
        first = torch.cumsum(take, 0) - take
        elem = starts_s[row_of] + (torch.arange(int(take.sum()), device=dev) - first[row_of])
        payload = data.to(dev).reshape(-1)[elem] if elem.numel() else data.to(dev).reshape(-1)[:0]
        row_owner = dest[order]
        send_elems = [int(take[row_owner == r].sum()) for r in range(self.P)]
        recv_rows = self.comm.exchange_counts(send_rows, dev)
        recv_elems = self.comm.exchange_counts(send_elems, dev)
        got_idx = self.comm.all_to_all(local_idx[order].to(torch.int32), send_rows, recv_rows)
        got_len = self.comm.all_to_all(lens_s.to(torch.int32), send_rows, recv_rows)
        got_data = self.comm.all_to_all(_as_bytes(payload), [e * esz for e in send_elems],
                                        [e * esz for e in recv_elems]).view(dtype)
        if got_idx.numel() == 0:
            return
        if ragged:
            got_cu = torch.zeros(got_len.numel() + 1, dtype=torch.int64, device=dev)
            got_cu[1:] = torch.cumsum(got_len.to(torch.int64), 0)
            self.local.put(column, got_idx, got_cu.to(torch.int32), got_data)
        else:
            self.local.put(column, got_idx, None, got_data)

    # -- the metadata broadcast ------------------------------------------------------------------
    def sync(self) -> None:
        """Collective: every rank's status words and claim bits to every rank."""
        parts = self.comm.all_gather_padded(self.local.status_words().to(self.device).to(torch.int32), self._n_local)
        for r, p in enumerate(parts):
            self.status[self._glob_samples[r]] = p
        for c in range(len(self.consumers)):
            bits = self.comm.all_gather_padded(self.local.claim_bits(c).to(self.device).to(torch.uint8), self._g_local)
            for r, b in enumerate(bits):
                self.claimed[c, self._glob_groups[r]] = b.to(torch.bool)

    # -- workflow steps 1 and 2, consumer side ------------------------------------------------
    def select(self, consumer: int, max_samples: int) -> torch.Tensor:
        """The global groups a get of `max_samples` serves now, ascending, from the replica."""
        need = self.consumers[consumer][0]
        ready = ((self.status & need) == need).view(self.map.G, self.map.N).all(dim=1) & ~self.claimed[consumer]
        return torch.nonzero(ready).reshape(-1)[:max_samples // self.map.N]

    def get(self, consumer: int, max_samples: int, home: Optional[int] = None) -> Optional[ShardedBatch]:
        """Collective.  Returns the batch on the home rank, None on the others."""
        m, dev = self.map, self.device
        if max_samples // m.N == 0:
            raise ValueError("max_samples holds no whole group")
        home = self.home_of(consumer) if home is None else home
        sel = self.select(consumer, max_samples)
        owner = m.owner_of_group(sel)
        k = [int((owner == r).sum()) for r in range(self.P)]                # groups per rank
        mine = sel[owner == self.rank]
        batch = self.local.get(consumer, k[self.rank] * m.N) if k[self.rank] else None
        n_mine = batch.n_samples if batch is not None else 0
        if n_mine != k[self.rank] * m.N or (n_mine and not torch.equal(
                m.global_sample(self.rank, batch.indices.to(dev).to(torch.int64))[::m.N] // m.N, mine)):
            raise RuntimeError("the local dock served other groups than the replica foresaw: a put ran "
                               "between the metadata broadcast and this get")
        self.claimed[consumer, sel] = True
        # lengths and advantages first (the home rank sizes its buffers from them), then the columns
        need_mask, out_mask, adv = self.consumers[consumer]
        n_r = [g * m.N for g in k]
        to_home = lambda n: [n if r == home else 0 for r in range(self.P)]
        from_all = lambda per: per if self.rank == home else [0] * self.P

        def send_home(x: torch.Tensor, per_rank: List[int]) -> torch.Tensor:
            return self.comm.all_to_all(x, to_home(x.numel()), from_all(per_rank))

        if batch is not None:
            lp = (batch.cu_prompt[1:] - batch.cu_prompt[:-1]).to(dev).to(torch.int32)
            lr = (batch.cu_response[1:] - batch.cu_response[:-1]).to(dev).to(torch.int32)
        else:
            lp = lr = torch.zeros(0, dtype=torch.int32, device=dev)
        all_lp, all_lr = send_home(lp, n_r), send_home(lr, n_r)
        all_adv = None
        if adv:
            a = batch.advantages.to(dev) if batch is not None else torch.zeros(0, dtype=torch.float32, device=dev)
            all_adv = send_home(a, n_r)
        tok_p = [0] * self.P
        tok_r = [0] * self.P
        if self.rank == home:
            off = 0
            for r in range(self.P):
                tok_p[r] = int(all_lp[off:off + n_r[r]].sum())
                tok_r[r] = int(all_lr[off:off + n_r[r]].sum())
                off += n_r[r]
        received: Dict[int, torch.Tensor] = {}
        for c, (dt, cls, _pad) in enumerate(self.columns):
            if not (out_mask >> c) & 1:
                continue
            dtype, esz = self.ELEM[dt]
            per = n_r if cls == "scalar" else (tok_p if cls == "prompt" else tok_r)
            mine_col = batch.columns[c].to(dev) if batch is not None else torch.zeros(0, dtype=dtype, device=dev)
            received[c] = send_home(_as_bytes(mine_col), [e * esz for e in per]).view(dtype)
        if self.rank != home:
            return None
        return self._assemble(consumer, sel, owner, k, n_r, all_lp, all_lr, all_adv, received, tok_p, tok_r)

    def _assemble(self, consumer, sel, owner, k, n_r, all_lp, all_lr, all_adv, received, tok_p, tok_r) -> ShardedBatch:
        """Home rank: the ranks' parts, each in its own (ascending) order, laid out in global group order."""
        m, dev = self.map, self.device
        n_total = int(sel.numel()) * m.N
        # position of every sample of the final batch inside the concatenation of the ranks' parts
        base = [0] * self.P
        for r in range(1, self.P):
            base[r] = base[r - 1] + n_r[r - 1]
        rank_pos = torch.zeros(sel.numel(), dtype=torch.int64, device=dev)          # group's place within its rank's part
        for r in range(self.P):
            sel_r = owner == r
            rank_pos[sel_r] = torch.arange(int(sel_r.sum()), device=dev)
        grp_src = torch.tensor(base, device=dev)[owner] + rank_pos * m.N           # first sample of each group, in arrival order
        src = (grp_src[:, None] + torch.arange(m.N, device=dev)[None, :]).reshape(-1)
        lp, lr = all_lp[src].to(torch.int64), all_lr[src].to(torch.int64)
        cu_p = torch.zeros(n_total + 1, dtype=torch.int64, device=dev)
        cu_r = torch.zeros(n_total + 1, dtype=torch.int64, device=dev)
        cu_p[1:], cu_r[1:] = torch.cumsum(lp, 0), torch.cumsum(lr, 0)
        # where each sample's rows start in the arrival buffers: per rank, prefix sums of its own lengths
        arr_p = torch.cumsum(all_lp.to(torch.int64), 0) - all_lp
        arr_r = torch.cumsum(all_lr.to(torch.int64), 0) - all_lr
        cols: Dict[int, torch.Tensor] = {}
        for c, buf in received.items():
            cls = self.columns[c][1]
            if cls == "scalar":
                cols[c] = buf[src]
                continue
            ln, arr = (lp, arr_p) if cls == "prompt" else (lr, arr_r)
            row_of = torch.repeat_interleave(torch.arange(n_total, device=dev), ln)
            first = torch.cumsum(ln, 0) - ln
            elem = arr[src][row_of] + (torch.arange(int(ln.sum()), device=dev) - first[row_of])
            cols[c] = buf[elem] if elem.numel() else buf[:0]
        indices = (sel[:, None] * m.N + torch.arange(m.N, device=dev)[None, :]).reshape(-1).to(torch.int32)
        return ShardedBatch(n_samples=n_total, n_groups=int(sel.numel()), indices=indices,
                            cu_prompt=cu_p.to(torch.int32), cu_response=cu_r.to(torch.int32),
                            cu_seq=(cu_p + cu_r).to(torch.int32), columns=cols,
                            advantages=all_adv[src] if all_adv is not None else None,
                            prompt_tokens=int(cu_p[-1]), response_tokens=int(cu_r[-1]))

    def reset(self) -> None:
        self.local.reset()
        self.status.zero_()
        self.claimed.zero_()


# --------------------------------------------------------------------------- the CUDA dock as a rank's local dock
class CudaLocal:
    """This rank's own dock: the C-ABI library through its binding.  max_prompt_len /
    max_response_len bound a row, so that output buffers for a get can be sized."""

    def __init__(self, smap: ShardMap, rank: int, columns: Sequence, consumers: Sequence, prompt_cap: int,
                 response_cap: int, reward_column: int, max_prompt_len: int, max_response_len: int,
                 eps: float = 1e-6, device: int = 0):
        from . import binding as td
        self.td = td
        g_local, s_local = smap.local_shape(rank)
        self.N = smap.N
        self.dock = td.Dock(g_local, smap.N, s_local, columns, consumers, prompt_cap, response_cap, reward_column, eps, device)
        self.device = self.dock.device
        self.max_p, self.max_r = max_prompt_len, max_response_len
        self._bufs: Dict = {}
        self._keep: List = []

    def put(self, column, indices, cu, data):
        self.dock.put(column, indices.contiguous(), cu.contiguous() if cu is not None else None, data.contiguous())
        self._keep.append((indices, cu, data))
        if len(self._keep) > 32:
            torch.cuda.current_stream().synchronize()
            self._keep.clear()

    def get(self, consumer: int, max_samples: int) -> LocalBatch:
        td = self.td
        key = (consumer, max_samples)
        if key not in self._bufs:
            self._bufs[key] = td.GetBuffers(self.dock, consumer, max_samples, td.PACKED,
                                            prompt_tokens_cap=max_samples * self.max_p,
                                            response_tokens_cap=max_samples * self.max_r)
        b = self._bufs[key]
        self.dock.get(b)
        res = b.read_result()
        if res.status:
            raise RuntimeError(f"local get reported status {res.status:#x}")
        n = res.n_samples
        cols = {}
        for c, t in b.cols.items():
            cls = self.dock.columns[c][1]
            tot = n if cls == td.SCALAR else (res.prompt_tokens if cls == td.PROMPT else res.response_tokens)
            cols[c] = t[:tot]
        return LocalBatch(n, b.indices[:n], b.cu_prompt[:n + 1], b.cu_response[:n + 1], cols,
                          b.advantages[:n] if b.advantages is not None else None)

    def status_words(self) -> torch.Tensor:
        torch.cuda.current_stream().synchronize()
        return self.dock.table(0).view(torch.int32).clone()

    def claim_bits(self, consumer: int) -> torch.Tensor:
        words = self.dock.table(4, consumer).view(torch.int32).clone().to(torch.int64) & 0xFFFFFFFF
        bits = (words[:, None] >> torch.arange(32, device=words.device)[None, :]) & 1
        return bits.reshape(-1)[:self.dock.G].to(torch.bool)

    def reset(self):
        self.dock.reset()
