"""Seeded synthetic GRPO sample-flow workloads.

This module only *draws inputs*: sample lengths, token ids, per-token
log-probabilities, rewards, and the order in which producers put columns and
consumers ask for batches.  It holds none of the transfer dock's arithmetic
(no selection, no offsets, no advantages), so that the CPU oracle and the CUDA
library can both be fed from it without sharing any of the method.

The paper's own runs use DeepScaleR prompts and model-generated responses
(Evaluation, "Experiment Setup"); neither is available offline, so the length
distributions below stand in for them.  Record schema follows the text under
Eq. 1: one prompt-length item, several response-length items, a few scalars.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

# dtype tags used across the repository (value = element size in bytes)
DTYPE_SIZE = {"i32": 4, "f32": 4, "bf16": 2}
DTYPE_NUMPY = {"i32": np.int32, "f32": np.float32, "bf16": np.uint16}

SCALAR, PROMPT, RESPONSE = "scalar", "prompt", "response"

BASE_SEED = 20250719


@dataclass(frozen=True)
class ColumnSpec:
    name: str
    dtype: str          # "i32" | "f32" | "bf16"
    cls: str            # SCALAR | PROMPT | RESPONSE
    pad_bits: int = 0   # raw bit pattern written into right-padding


@dataclass(frozen=True)
class ConsumerSpec:
    name: str
    need: Tuple[str, ...]   # columns that must be ready before a sample is served
    out: Tuple[str, ...]    # columns gathered into the batch
    advantage: bool = False


@dataclass
class Op:
    """One call of a schedule: a put of `column` for `indices`, or a get."""
    kind: str                         # "put" | "get" | "put_back" | "get_many" | "put_back_many"
    column: int = -1                  # put: column number
    indices: Optional[np.ndarray] = None  # put: int32 sample indices, call order
    consumer: int = -1                # get: consumer number
    max_samples: int = 0              # get: micro-batch size
    columns: Optional[List[int]] = None   # put_back: columns `consumer` sends back for the batch it got last
    group: Optional[List] = None          # get_many: consumers served by one call, in order (one micro-batch each);
                                          # put_back_many: (consumer, column) pairs sent back by one call, in order


@dataclass
class Workload:
    name: str
    config_id: int
    G: int                      # prompts
    N: int                      # responses per prompt
    S: int                      # warehouse shards
    columns: List[ColumnSpec]
    consumers: List[ConsumerSpec]
    micro_batch: int            # samples per get
    len_prompt: np.ndarray      # int32 [n]
    len_response: np.ndarray    # int32 [n]
    data: Dict[str, np.ndarray]  # column -> rows concatenated in index order
    pad_prompt_to: int
    pad_response_to: int
    vocab: int
    seed: int
    ops: List[Op] = field(default_factory=list)
    # cascade schedule: column -> what a worker state sends back for a batch, rows packed in batch
    # order (row i of the batch at cu[i]); long enough for the largest micro-batch
    pool: Dict[int, np.ndarray] = field(default_factory=dict)

    @property
    def n(self) -> int:
        return self.G * self.N

    def column_index(self, name: str) -> int:
        for i, c in enumerate(self.columns):
            if c.name == name:
                return i
        raise KeyError(name)

    def lengths(self, cls: str) -> np.ndarray:
        return self.len_prompt if cls == PROMPT else self.len_response

    def row_starts(self, cls: str) -> np.ndarray:
        """int64 [n+1] start of each sample's row inside `data[col]` (index order)."""
        out = np.zeros(self.n + 1, dtype=np.int64)
        np.cumsum(self.lengths(cls), out=out[1:])
        return out

    def mask(self, names: Sequence[str]) -> int:
        m = 0
        for nm in names:
            m |= 1 << self.column_index(nm)
        return m

    def pack(self, column: int, indices: np.ndarray) -> Tuple[Optional[np.ndarray], np.ndarray]:
        """Producer-side packing of one put call: rows of `indices`, in that order,
        concatenated; returns (cu int32 [k+1] or None for a scalar column, data)."""
        spec = self.columns[column]
        src = self.data[spec.name]
        idx = np.asarray(indices, dtype=np.int64)
        if spec.cls == SCALAR:
            return None, np.ascontiguousarray(src[idx])
        starts = self.row_starts(spec.cls)
        lens = self.lengths(spec.cls)[idx].astype(np.int64)
        cu = np.zeros(len(idx) + 1, dtype=np.int64)
        np.cumsum(lens, out=cu[1:])
        assert cu[-1] < 2 ** 31, "one put call must hold fewer than 2^31 elements"
        out = np.empty(int(cu[-1]), dtype=src.dtype)
        if len(idx) and np.all(np.diff(idx) == 1):
            out[:] = src[starts[idx[0]]:starts[idx[-1] + 1]]
        else:
            for j, s in enumerate(idx):
                out[cu[j]:cu[j + 1]] = src[starts[s]:starts[s + 1]]
        return cu.astype(np.int32), out

    def column_tuples(self) -> List[Tuple[str, str, int]]:
        return [(c.dtype, c.cls, c.pad_bits) for c in self.columns]

    def consumer_tuples(self) -> List[Tuple[int, int, bool]]:
        return [(self.mask(k.need), self.mask(k.out), k.advantage) for k in self.consumers]

    def shard_capacity(self, cls: str) -> int:
        """A generous per-shard arena size in elements: every row of the fullest
        shard plus eight spare elements per row for alignment padding."""
        per = (self.lengths(cls).astype(np.int64) + 8).reshape(self.S, -1).sum(axis=1)
        return int(per.max())

    def tokens_total(self) -> int:
        return int(self.len_prompt.sum(dtype=np.int64) + self.len_response.sum(dtype=np.int64))

    def payload_bytes(self) -> int:
        """Bytes of all columns of all samples (one copy)."""
        return int(sum(a.nbytes for a in self.data.values()))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of finite float32 values to bf16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = u + 0x7FFF + ((u >> 16) & 1)
    return (rounded >> 16).astype(np.uint16)


def standard_columns(with_entropy: bool = False) -> List[ColumnSpec]:
    cols = [
        ColumnSpec("prompt_ids", "i32", PROMPT),
        ColumnSpec("response_ids", "i32", RESPONSE),
        ColumnSpec("old_logprob", "f32", RESPONSE),
        ColumnSpec("ref_logprob", "f32", RESPONSE),
        ColumnSpec("reward", "f32", SCALAR),
    ]
    if with_entropy:
        cols.append(ColumnSpec("entropy", "bf16", RESPONSE))
    return cols


def standard_consumers(columns: Sequence[ColumnSpec]) -> List[ConsumerSpec]:
    ids = ("prompt_ids", "response_ids")
    everything = tuple(c.name for c in columns)
    return [
        ConsumerSpec("reference", ids, ids),
        ConsumerSpec("reward", ids, ids),
        ConsumerSpec("actor_inference", ids, ids),
        ConsumerSpec("actor_update", everything, everything, advantage=True),
    ]


def _lognormal_lengths(rng: np.random.Generator, size: int, median: float, sigma: float, cap: int) -> np.ndarray:
    x = rng.lognormal(mean=np.log(median), sigma=sigma, size=size)
    return np.clip(np.rint(x), 1, cap).astype(np.int32)


def _draw_data(rng: np.random.Generator, columns: Sequence[ColumnSpec], len_p: np.ndarray,
               len_r: np.ndarray, vocab: int) -> Dict[str, np.ndarray]:
    n = len(len_p)
    tot = {PROMPT: int(len_p.sum(dtype=np.int64)), RESPONSE: int(len_r.sum(dtype=np.int64)), SCALAR: n}
    data: Dict[str, np.ndarray] = {}
    for c in columns:
        m = tot[c.cls]
        if c.name == "reward":
            data[c.name] = rng.standard_normal(m, dtype=np.float32)
        elif c.dtype == "i32":
            data[c.name] = rng.integers(0, vocab, size=m, dtype=np.int32)
        elif c.dtype == "f32":
            a = rng.random(m, dtype=np.float32)
            a *= np.float32(10.0)
            a -= np.float32(10.0)           # uniform on [-10, 0)
            data[c.name] = a
        elif c.dtype == "bf16":
            a = rng.random(m, dtype=np.float32)
            a *= np.float32(4.0)            # uniform on [0, 4)
            data[c.name] = f32_to_bf16_bits(a)
        else:
            raise ValueError(c.dtype)
    return data


def _chunks(rng: np.random.Generator, order: np.ndarray, lo: int, hi: int) -> List[np.ndarray]:
    out, p = [], 0
    while p < len(order):
        k = int(rng.integers(lo, hi + 1))
        out.append(order[p:p + k].astype(np.int32))
        p += k
    return out


def _bulk_ops(w: Workload) -> List[Op]:
    """One put per column over all samples in index order, then round-robin gets
    that drain every consumer exactly."""
    ops = [Op("put", column=c, indices=np.arange(w.n, dtype=np.int32)) for c in range(len(w.columns))]
    rounds = -(-w.n // w.micro_batch)
    for _ in range(rounds):
        for c in range(len(w.consumers)):
            ops.append(Op("get", consumer=c, max_samples=w.micro_batch))
    return ops


def _random_order_ops(w: Workload, rng: np.random.Generator, lo: int, hi: int) -> List[Op]:
    """Every column put in its own seeded random sample order in chunks of lo..hi
    samples, all before the first get; then round-robin gets until drained."""
    puts: List[Op] = []
    for c in range(len(w.columns)):
        for ch in _chunks(rng, rng.permutation(w.n), lo, hi):
            puts.append(Op("put", column=c, indices=ch))
    perm = rng.permutation(len(puts))
    ops = [puts[i] for i in perm]
    rounds = -(-w.n // w.micro_batch)
    for _ in range(rounds):
        for c in range(len(w.consumers)):
            ops.append(Op("get", consumer=c, max_samples=w.micro_batch))
    return ops


def _interleaved_ops(w: Workload, rng: np.random.Generator, lo: int, hi: int, poll_every: int) -> List[Op]:
    """Out-of-order readiness: shuffled put chunks with every consumer polling after
    each `poll_every` puts, so that gets meet partially ready docks.  The trailing
    polls are enough to drain whatever an in-order execution left behind."""
    puts: List[Op] = []
    for c in range(len(w.columns)):
        for ch in _chunks(rng, rng.permutation(w.n), lo, hi):
            puts.append(Op("put", column=c, indices=ch))
    perm = rng.permutation(len(puts))
    ops: List[Op] = []
    for j, i in enumerate(perm):
        ops.append(puts[i])
        if (j + 1) % poll_every == 0:
            for c in range(len(w.consumers)):
                ops.append(Op("get", consumer=c, max_samples=w.micro_batch))
    rounds = -(-w.n // w.micro_batch)
    for _ in range(rounds):
        for c in range(len(w.consumers)):
            ops.append(Op("get", consumer=c, max_samples=w.micro_batch))
    return ops


# Which worker state produces which column in the cascade (Fig. 1: the inference states feed the
# actor update): the reference model its log-probs, the reward state the reward, the actor's
# inference pass the old log-probs (and the entropy, where the shape has it).
CASCADE_PRODUCES = {"reference": ("ref_logprob",), "reward": ("reward",),
                    "actor_inference": ("old_logprob", "entropy")}


def _cascade_ops(w: Workload, rng: np.random.Generator, lo: int, hi: int, poll_every: int,
                 batched: bool = False) -> List[Op]:
    """The whole sample flow on one dock: generation puts prompt and response ids in shuffled
    chunks; every `poll_every` puts each inference state takes a micro-batch and sends its
    column back for exactly that batch, and the actor update takes what has become complete.
    batched: a poll is one get call for all worker states together and one write-back call for
    all of them (the actor update then sees a poll's write-backs at the next poll)."""
    gen = [w.column_index("prompt_ids"), w.column_index("response_ids")]
    names = [c.name for c in w.columns]
    produces = {ci: [w.column_index(nm) for nm in CASCADE_PRODUCES.get(k.name, ()) if nm in names]
                for ci, k in enumerate(w.consumers)}
    # the pools: seeded values of each produced column's type, sized for the largest micro-batch
    top_r = int(np.sort(w.len_response)[::-1][:w.micro_batch].sum(dtype=np.int64))
    for cols in produces.values():
        for c in cols:
            spec = w.columns[c]
            m = w.micro_batch if spec.cls == SCALAR else top_r
            if spec.name == "reward":
                w.pool[c] = rng.standard_normal(m, dtype=np.float32)
            elif spec.dtype == "bf16":
                w.pool[c] = f32_to_bf16_bits(rng.random(m, dtype=np.float32) * np.float32(4.0))
            else:
                w.pool[c] = (rng.random(m, dtype=np.float32) * np.float32(10.0) - np.float32(10.0)).astype(np.float32)
    puts: List[Op] = []
    for c in gen:
        for ch in _chunks(rng, rng.permutation(w.n), lo, hi):
            puts.append(Op("put", column=c, indices=ch))
    workers = [ci for ci, cols in produces.items() if cols]
    updaters = [ci for ci, cols in produces.items() if not cols]

    def poll(ops: List[Op], inference: bool = True):
        if batched:
            ops.append(Op("get_many", group=(workers if inference else []) + updaters, max_samples=w.micro_batch))
            if inference:
                ops.append(Op("put_back_many", group=[(ci, c) for ci in workers for c in produces[ci]]))
            return
        if inference:
            for ci in workers:
                ops.append(Op("get", consumer=ci, max_samples=w.micro_batch))
                ops.append(Op("put_back", consumer=ci, columns=produces[ci]))
        for ci in updaters:
            ops.append(Op("get", consumer=ci, max_samples=w.micro_batch))

    ops: List[Op] = []
    for j, i in enumerate(rng.permutation(len(puts))):
        ops.append(puts[i])
        if (j + 1) % poll_every == 0:
            poll(ops)
    rounds = -(-w.n // w.micro_batch)
    for _ in range(rounds):
        poll(ops)
    for _ in range(rounds):
        poll(ops, inference=False)
    return ops


def make_custom(name: str, G: int, N: int, S: int, *, prompt_len: Tuple[int, int],
                response: Tuple, vocab: int, micro_batch: int, seed: int,
                with_entropy: bool = False, schedule: str = "bulk",
                chunk: Tuple[int, int] = (1, 16), poll_every: int = 8,
                config_id: int = 0, pad_prompt_to: Optional[int] = None,
                pad_response_to: Optional[int] = None) -> Workload:
    """response = ("uniform", lo, hi) or ("lognormal", median, sigma, cap)."""
    assert G % S == 0, "shards hold whole prompts: S must divide G"
    rng = np.random.Generator(np.random.PCG64(seed))
    per_prompt = rng.integers(prompt_len[0], prompt_len[1] + 1, size=G, dtype=np.int32)
    len_p = np.repeat(per_prompt, N).astype(np.int32)
    if response[0] == "uniform":
        len_r = rng.integers(response[1], response[2] + 1, size=G * N, dtype=np.int32)
        cap_r = response[2]
    else:
        _, median, sigma, cap_r = response
        len_r = _lognormal_lengths(rng, G * N, median, sigma, cap_r)
    cols = standard_columns(with_entropy)
    data = _draw_data(rng, cols, len_p, len_r, vocab)
    w = Workload(name=name, config_id=config_id, G=G, N=N, S=S, columns=cols,
                 consumers=standard_consumers(cols), micro_batch=micro_batch,
                 len_prompt=len_p, len_response=len_r, data=data,
                 pad_prompt_to=pad_prompt_to or prompt_len[1],
                 pad_response_to=pad_response_to or cap_r, vocab=vocab, seed=seed)
    if schedule == "bulk":
        w.ops = _bulk_ops(w)
    elif schedule == "random_order":
        w.ops = _random_order_ops(w, rng, *chunk)
    elif schedule == "interleaved":
        w.ops = _interleaved_ops(w, rng, chunk[0], chunk[1], poll_every)
    elif schedule in ("cascade", "cascade_batched"):
        w.ops = _cascade_ops(w, rng, chunk[0], chunk[1], poll_every, batched=schedule == "cascade_batched")
    elif schedule == "none":
        w.ops = []
    else:
        raise ValueError(schedule)
    return w


SIGMA_HEADLINE = 0.25   # spread of the lognormal response lengths

CONFIG_NAMES = {
    1: "tiny-grpo-64",
    2: "qwen2.5-7b-shaped-2048",
    3: "qwen2.5-32b-shaped-8192",
    4: "qwen3-30b-moe-shaped-out-of-order-16384",
    5: "deepseek-r1-671b-shaped-12288",
}


def make_config(config_id: int, seed: Optional[int] = None, sigma: float = SIGMA_HEADLINE,
                schedule: Optional[str] = None) -> Workload:
    """The five benchmark shapes.  `schedule` overrides the default call order ("cascade":
    generation chunks of a quarter to four micro-batches, a poll every four puts)."""
    seed = BASE_SEED + config_id if seed is None else seed
    name = CONFIG_NAMES[config_id]
    if schedule in ("cascade", "cascade_batched"):
        base = make_config(config_id, seed, sigma, "none")
        spec = {1: ((16, 64), ("uniform", 32, 256), 151936), 2: ((128, 1024), ("lognormal", 1500.0, sigma, 4096), 152064),
                3: ((256, 2048), ("lognormal", 3000.0, sigma, 16384), 152064),
                4: ((256, 2048), ("lognormal", 2500.0, sigma, 8192), 151936),
                5: ((512, 4096), ("lognormal", 6000.0, sigma, 32768), 129280)}[config_id]
        mb = base.micro_batch
        return make_custom(name + "-cascade", base.G, base.N, base.S, prompt_len=spec[0], response=spec[1],
                           vocab=spec[2], micro_batch=mb, seed=seed, with_entropy=config_id == 3,
                           schedule=schedule, chunk=(max(mb // 4, 1), mb * 4), poll_every=4,
                           config_id=config_id)
    if config_id == 1:
        return make_custom(name, 16, 4, 2, prompt_len=(16, 64), response=("uniform", 32, 256),
                           vocab=151936, micro_batch=8, seed=seed,
                           schedule=schedule or "random_order", chunk=(1, 16), config_id=1)
    if config_id == 2:
        return make_custom(name, 256, 8, 4, prompt_len=(128, 1024),
                           response=("lognormal", 1500.0, sigma, 4096), vocab=152064,
                           micro_batch=64, seed=seed, schedule=schedule or "bulk", config_id=2)
    if config_id == 3:
        return make_custom(name, 512, 16, 8, prompt_len=(256, 2048),
                           response=("lognormal", 3000.0, sigma, 16384), vocab=152064,
                           micro_batch=128, seed=seed, with_entropy=True,
                           schedule=schedule or "bulk", config_id=3)
    if config_id == 4:
        return make_custom(name, 1024, 16, 16, prompt_len=(256, 2048),
                           response=("lognormal", 2500.0, sigma, 8192), vocab=151936,
                           micro_batch=128, seed=seed, schedule=schedule or "interleaved",
                           chunk=(1, 64), poll_every=8, config_id=4)
    if config_id == 5:
        return make_custom(name, 384, 32, 16, prompt_len=(512, 4096),
                           response=("lognormal", 6000.0, sigma, 32768), vocab=129280,
                           micro_batch=256, seed=seed, schedule=schedule or "bulk", config_id=5)
    raise ValueError(f"no config {config_id}")
