"""Pins for the CPU oracle's put/get: every expected value below comes from the
generator's own arrays, from numpy library routines, from closed forms or from
brute force, never from the oracle itself or from the CUDA path."""
import itertools

import numpy as np
import pytest

from oracle import td_oracle as ora
from paper_2507_19017_b200 import workloads as wl
from tests import helpers as H


def small(schedule="random_order", **kw):
    args = dict(G=8, N=4, S=2, prompt_len=(3, 40), response=("uniform", 1, 90), vocab=1000,
                micro_batch=8, seed=7, schedule=schedule, chunk=(1, 5))
    args.update(kw)
    return wl.make_custom("small", **args)


# ---------------------------------------------------------------- round trip
@pytest.mark.parametrize("entropy", [False, True])
def test_identity_round_trip_packed(entropy):
    """Put every column in a random order and chunking, then one get of everything:
    each packed output is the generator's array, rows in index order."""
    w = small(with_entropy=entropy)
    d = H.make_oracle(w)
    for op in w.ops:
        if op.kind == "put":
            cu, data = w.pack(op.column, op.indices)
            assert d.put(op.column, op.indices, cu, data) == len(op.indices)
    upd = len(w.consumers) - 1
    b = d.get(upd, w.n)
    assert b.n_samples == w.n and b.n_groups == w.G and b.status == 0
    assert np.array_equal(b.indices, np.arange(w.n))
    for c, spec in enumerate(w.columns):
        assert H.bits_equal(b.columns[c], w.data[spec.name]), spec.name
    assert b.prompt_tokens == int(w.len_prompt.sum()) and b.response_tokens == int(w.len_response.sum())


def test_identity_round_trip_padded():
    w = small()
    d = H.make_oracle(w)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, np.arange(w.n, dtype=np.int32))
        d.put(c, np.arange(w.n), cu, data)
    b = d.get(3, w.n, ora.PADDED, 40, 96)
    idx = np.arange(w.n)
    for c, spec in enumerate(w.columns):
        if spec.cls == wl.SCALAR:
            assert H.bits_equal(b.columns[c], w.data[spec.name])
        else:
            width = 40 if spec.cls == wl.PROMPT else 96
            assert H.bits_equal(b.columns[c], H.expected_padded(w, c, idx, width)), spec.name


def test_identity_round_trip_left_padded_prompts():
    """Prompt rows flush right in their width (the pad in front), response rows as before:
    expected values from the generator's arrays; the flag changes nothing else of the batch."""
    w = small(with_entropy=True)
    d = H.make_oracle(w)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, np.arange(w.n, dtype=np.int32))
        d.put(c, np.arange(w.n), cu, data)
    upd = len(w.consumers) - 1
    b = d.get(upd, w.n, ora.PADDED, 40, 96, out_flags=ora.OUT_LEFT_PAD_PROMPT)
    idx = np.arange(w.n)
    assert b.n_samples == w.n and b.status == 0
    assert np.array_equal(b.cu_prompt, np.concatenate(([0], np.cumsum(w.len_prompt))))
    for c, spec in enumerate(w.columns):
        if spec.cls == wl.SCALAR:
            assert H.bits_equal(b.columns[c], w.data[spec.name])
        else:
            width = 40 if spec.cls == wl.PROMPT else 96
            assert H.bits_equal(b.columns[c], H.expected_padded(w, c, idx, width, left=spec.cls == wl.PROMPT)), spec.name
    # a packed get ignores the flag; an unknown flag is refused
    g = d.gather(upd, idx[:8], out_flags=ora.OUT_LEFT_PAD_PROMPT)
    assert H.bits_equal(g.columns[0], w.pack(0, idx[:8].astype(np.int32))[1])
    with pytest.raises(ValueError):
        d.gather(upd, idx[:8], out_flags=2)


def test_left_padded_prompts_by_hand():
    cols = [("i32", "prompt", 0xDEADBEEF), ("bf16", "prompt", 0xABCD), ("f32", "response", 0x7FC00001)]
    d = ora.OracleDock(1, 3, 1, cols, [(0x7, 0x7, False)], 64, 64, 0)
    d.put(0, [0, 1, 2], np.array([0, 2, 2, 5], np.int32), np.array([5, 6, 7, 8, 9], np.int32))
    d.put(1, [0, 1, 2], np.array([0, 2, 2, 5], np.int32), np.array([1, 2, 3, 4, 5], np.uint16))
    d.put(2, [0, 1, 2], np.array([0, 1, 3, 3], np.int32), np.array([1, 2, 3], np.float32))
    b = d.get(0, 3, ora.PADDED, 3, 2, out_flags=ora.OUT_LEFT_PAD_PROMPT)
    P = 0xDEADBEEF
    assert b.columns[0].view(np.uint32).tolist() == [[P, 5, 6], [P, P, P], [7, 8, 9]]      # widths 2, 0 and 3 of 3
    assert b.columns[1].tolist() == [[0xABCD, 1, 2], [0xABCD] * 3, [3, 4, 5]]
    assert b.columns[2].view(np.uint32).tolist() == [[0x3F800000, 0x7FC00001], [0x40000000, 0x40400000],
                                                     [0x7FC00001, 0x7FC00001]]               # responses: pad behind


def test_padded_uses_the_columns_pad_bits():
    cols = [("i32", "prompt", 0xDEADBEEF), ("f32", "response", 0x7FC00001), ("bf16", "response", 0xABCD),
            ("f32", "scalar", 0)]
    d = ora.OracleDock(1, 2, 1, cols, [(0xF, 0xF, True)], 64, 64, 3)
    d.put(0, [0, 1], np.array([0, 2, 3], np.int32), np.array([5, 6, 7], np.int32))
    d.put(1, [0, 1], np.array([0, 1, 4], np.int32), np.array([1, 2, 3, 4], np.float32))
    d.put(2, [0, 1], np.array([0, 1, 4], np.int32), np.array([9, 8, 7, 6], np.uint16))
    d.put(3, [0, 1], None, np.array([0.5, 1.5], np.float32))
    b = d.get(0, 2, ora.PADDED, 3, 4)
    assert b.columns[0].view(np.uint32).tolist() == [[5, 6, 0xDEADBEEF], [7, 0xDEADBEEF, 0xDEADBEEF]]
    assert b.columns[1].view(np.uint32)[0].tolist() == [0x3F800000, 0x7FC00001, 0x7FC00001, 0x7FC00001]
    assert b.columns[2].tolist() == [[9, 0xABCD, 0xABCD, 0xABCD], [8, 7, 6, 0xABCD]]


def test_payload_bits_survive_nan_and_negative_zero():
    cols = [("f32", "response", 0), ("f32", "scalar", 0)]
    d = ora.OracleDock(1, 1, 1, cols, [(3, 3, False)], 8, 8, 1)
    weird = np.array([0x7FC01234, 0x80000000, 0xFF800000, 0x00000001], np.uint32)
    d.put(0, [0], np.array([0, 4], np.int32), weird.view(np.float32))
    d.put(1, [0], None, np.array([0xFFC00000], np.uint32).view(np.float32))
    b = d.get(0, 1)
    assert b.columns[0].view(np.uint32).tolist() == weird.tolist()
    assert b.columns[1].view(np.uint32).tolist() == [0xFFC00000]


# ------------------------------------------------------ selection / dispatch
def test_every_sample_dispatched_exactly_once_per_consumer():
    w = wl.make_config(1)
    d = H.make_oracle(w)
    batches = H.replay_oracle(w, d)
    seen = {c: [] for c in range(len(w.consumers))}
    for c, b in batches:
        assert b.n_samples % w.N == 0 and b.n_samples <= w.micro_batch
        assert np.all(np.diff(b.indices) > 0)                       # ascending
        grp = b.indices.reshape(-1, w.N)
        assert np.array_equal(grp, grp[:, :1] + np.arange(w.N))     # whole groups
        assert np.all(grp[:, 0] % w.N == 0)
        seen[c].extend(b.indices.tolist())
    for c in seen:
        assert sorted(seen[c]) == list(range(w.n))
        assert H.popcount_words(d.consumed_words(c)) == w.n
        assert H.popcount_words(d.claim_words(c)) == w.G
    # lowest index first: with everything ready, consumer batches come in index order
    for c in seen:
        assert seen[c] == list(range(w.n))
    # the dispatch counters say what this test saw dispatched: samples per consumer, and their
    # tokens counted from the generator's lengths
    st = d.stats()
    tokens = {c: 0 for c in seen}
    for c, b in batches:
        tokens[c] += int(w.len_prompt[b.indices].sum(dtype=np.int64) + w.len_response[b.indices].sum(dtype=np.int64))
    for c in seen:
        assert st.got_samples[c] == len(seen[c]) == w.n
        assert st.got_tokens[c] == tokens[c] == w.tokens_total()
    assert all(st.got_samples[c] == 0 and st.got_tokens[c] == 0 for c in range(len(w.consumers), 32))
    assert st.n_truncated == 0 and st.error_word == 0


def test_batches_match_generator_rows_and_cumsum():
    w = wl.make_config(1)
    d = H.make_oracle(w)
    for c, b in H.replay_oracle(w, d):
        lp, lr = w.len_prompt[b.indices], w.len_response[b.indices]
        assert np.array_equal(b.cu_prompt, np.concatenate([[0], np.cumsum(lp)]))
        assert np.array_equal(b.cu_response, np.concatenate([[0], np.cumsum(lr)]))
        assert np.array_equal(b.cu_seq, np.concatenate([[0], np.cumsum(lp + lr)]))
        assert b.prompt_tokens == lp.sum() and b.response_tokens == lr.sum()
        outm = w.consumer_tuples()[c][1]
        assert sorted(b.columns) == [k for k in range(len(w.columns)) if (outm >> k) & 1]
        for k, arr in b.columns.items():
            assert H.bits_equal(arr, H.expected_packed(w, k, b.indices))


def brute_force_select(status, need, claimed, G, N, m):
    """Definition: ready unclaimed groups, sorted, first m."""
    ready = [g for g in range(G)
             if not claimed[g] and all((status[g * N + j] & need) == need for j in range(N))]
    return sorted(ready)[:m]


@pytest.mark.parametrize("G,N", [(3, 2), (2, 3), (4, 1), (6, 1)])
def test_selection_brute_force_all_readiness_patterns(G, N):
    """Two columns, every subset of (sample, column) cells put; compare the groups a
    get returns with filter-sort-take over the same readiness table."""
    n = G * N
    cols = [("i32", "prompt", 0), ("f32", "scalar", 0)]
    cells = [(s, c) for s in range(n) for c in range(2)]
    assert len(cells) <= 12
    for pattern in range(1 << len(cells)):
        d = ora.OracleDock(G, N, 1, cols, [(3, 3, False), (1, 1, False)], 64, 64, 1)
        status = [0] * n
        for b, (s, c) in enumerate(cells):
            if (pattern >> b) & 1:
                if c == 0:
                    d.put(0, [s], np.array([0, 1], np.int32), np.array([s], np.int32))
                else:
                    d.put(1, [s], None, np.array([float(s)], np.float32))
                status[s] |= 1 << c
        assert d.status().tolist() == status
        for cons, need in ((0, 3), (1, 1)):
            claimed = [False] * G
            for m in (1, 2, G):
                want = brute_force_select(status, need, claimed, G, N, m)
                got = d.get(cons, m * N)
                assert got.indices.tolist() == [g * N + j for g in want for j in range(N)], (pattern, cons, m)
                for g in want:
                    claimed[g] = True
        d.close()


def test_partial_readiness_and_rounding_down():
    w = small(schedule="none", G=4, N=4, S=2)
    d = H.make_oracle(w)
    ids = [w.column_index("prompt_ids"), w.column_index("response_ids")]
    # only group 2 complete, group 0 lacks one sample
    for c in ids:
        for s in [8, 9, 10, 11, 0, 1, 2]:
            cu, data = w.pack(c, np.array([s], np.int32))
            d.put(c, [s], cu, data)
    b = d.get(0, 7)                     # 7 samples -> one group of 4
    assert b.indices.tolist() == [8, 9, 10, 11]
    assert d.get(0, 16).n_samples == 0  # nothing else ready: not an error
    for c in ids:
        cu, data = w.pack(c, np.array([3], np.int32))
        d.put(c, [3], cu, data)
    assert d.get(0, 16).indices.tolist() == [0, 1, 2, 3]
    # consumer 3 needs every column: still nothing
    assert d.get(3, 16).n_samples == 0
    with pytest.raises(ValueError):
        d.get(0, 3)                     # fewer than one group asked for


# ---------------------------------------------------------- offsets / arenas
def test_hand_computed_offsets():
    """G=3, N=2, S=3 (one prompt per shard).  Rows start on multiples of 8 elements,
    in arrival order per shard, and the first column of a class fixes the place."""
    cols = [("i32", "response", 0), ("f32", "response", 0), ("i32", "prompt", 0), ("f32", "scalar", 0)]
    d = ora.OracleDock(3, 2, 3, cols, [(0xF, 0xF, True)], 64, 64, 3)
    assert [d.shard_of(s) for s in range(6)] == [0, 0, 1, 1, 2, 2]
    # response column 1 arrives first for samples 5, 0, 1 with lengths 3, 9, 8
    d.put(1, [5, 0, 1], np.array([0, 3, 12, 20], np.int32), np.arange(20, dtype=np.float32))
    assert d.offsets(2).tolist() == [0, 16, -1, -1, -1, 0]
    assert d.lengths(2).tolist() == [9, 8, -1, -1, -1, 3]
    assert d.cursors(2).tolist() == [24, 0, 8]
    # column 0 for samples 1, 4, 0: 1 and 0 reuse their rows, 4 (length 0) takes no room
    d.put(0, [1, 4, 0], np.array([0, 8, 8, 17], np.int32), np.arange(17, dtype=np.int32))
    assert d.offsets(2).tolist() == [0, 16, -1, -1, 8, 0]
    assert d.lengths(2).tolist() == [9, 8, -1, -1, 0, 3]
    assert d.cursors(2).tolist() == [24, 0, 8]
    assert d.cursors(1).tolist() == [0, 0, 0]
    # payload landed where the offsets say
    a0 = d.arena(0, 0)
    assert a0[16:24].tolist() == list(range(0, 8)) and a0[0:9].tolist() == list(range(8, 17))
    a1 = d.arena(1, 0)
    assert a1[0:9].tolist() == list(range(3, 12)) and a1[16:24].tolist() == list(range(12, 20))
    assert d.arena(1, 2)[0:3].tolist() == [0, 1, 2]
    assert d.status().tolist() == [3, 3, 0, 0, 1, 2]


def test_offset_invariants_random_order():
    w = wl.make_config(1)
    d = H.make_oracle(w)
    H.replay_oracle(w, d)
    for cls, lens in ((1, w.len_prompt), (2, w.len_response)):
        off, ln = d.offsets(cls), d.lengths(cls)
        assert np.array_equal(ln, lens)
        assert np.all(off % 8 == 0)
        shard = np.array([d.shard_of(s) for s in range(w.n)])
        for sh in range(w.S):
            sel = np.where(shard == sh)[0]
            order = sel[np.argsort(off[sel])]
            ends = off[order] + (ln[order] + 7) // 8 * 8
            assert np.all(off[order][1:] == ends[:-1])          # rows tile the arena without gaps
            assert off[order][0] == 0 and ends[-1] == d.cursors(cls)[sh]
    st = d.status()
    assert np.all(st == (1 << len(w.columns)) - 1)
    for c in range(len(w.columns)):
        assert d.stats().put_accepted[c] == w.n


# ----------------------------------------------------------------- advantages
def test_advantages_against_numpy_and_closed_forms():
    w = wl.make_config(1)
    d = H.make_oracle(w)
    eps = float(np.float32(1e-6))
    for c, b in H.replay_oracle(w, d):
        if b.advantages is None:
            assert not w.consumers[c].advantage
            continue
        r = w.data["reward"][b.indices].astype(np.float64).reshape(-1, w.N)
        want = (r - r.mean(axis=1, keepdims=True)) / (r.std(axis=1, ddof=0, keepdims=True) + eps)
        got = b.advantages.astype(np.float64).reshape(-1, w.N)
        assert np.allclose(got, want, rtol=1e-6, atol=1e-7)
        assert np.all(np.abs(got.mean(axis=1)) <= 1e-6)
        sd = r.std(axis=1)
        assert np.allclose(got.std(axis=1), sd / (sd + eps), rtol=1e-6)


@pytest.mark.parametrize("N", [2, 3, 5, 7, 32])
def test_advantages_special_cases(N):
    cols = [("i32", "prompt", 0), ("f32", "scalar", 0)]
    G = 4
    d = ora.OracleDock(G, N, 1, cols, [(3, 3, True)], 8 * G * N, 8, 1, eps=1e-6)
    n = G * N
    rng = np.random.default_rng(N)
    rew = np.empty(n, np.float32)
    rew[0:N] = np.float32(0.3)                      # all equal (not exactly representable)
    rew[N:2 * N] = (np.arange(N) % 2).astype(np.float32)          # binary rule reward
    rew[2 * N:3 * N] = rng.standard_normal(N).astype(np.float32)
    rew[3 * N:] = np.float32(1e4) + rng.standard_normal(N).astype(np.float32) * np.float32(1e-3)
    d.put(0, np.arange(n), np.arange(n + 1, dtype=np.int32), np.zeros(n, np.int32))
    d.put(1, np.arange(n), None, rew)
    a = d.get(0, n).advantages.astype(np.float64).reshape(G, N)
    assert np.all(a[0] == 0.0)                      # zero variance -> exactly zero
    eps = float(np.float32(1e-6))
    r = rew.astype(np.float64).reshape(G, N)
    want = (r - r.mean(1, keepdims=True)) / (r.std(1, keepdims=True) + eps)
    assert np.allclose(a, want, rtol=1e-6, atol=1e-7)
    if N == 2:
        sd = np.abs(r[:, 0] - r[:, 1]) / 2
        z = sd / (sd + eps)
        assert np.allclose(np.abs(a[:, 0]), z, rtol=1e-6) and np.allclose(a[:, 0], -a[:, 1], rtol=1e-6)
        assert np.all(np.sign(a[1:, 0]) == np.sign(r[1:, 0] - r[1:, 1]))


# ------------------------------------------------------------------ error paths
def test_duplicate_oob_mismatch_and_bad_length_are_counted_and_skipped():
    w = small(schedule="none")
    d = H.make_oracle(w)
    rid, old = w.column_index("response_ids"), w.column_index("old_logprob")
    idx = np.array([0, 1, 2], np.int32)
    cu, data = w.pack(rid, idx)
    assert d.put(rid, idx, cu, data) == 3
    assert d.put(rid, np.array([1, -1, w.n, 3], np.int32),
                 *w.pack(rid, np.array([1, 0, 0, 3], np.int32))) == 1
    st = d.stats()
    assert (st.n_dup, st.n_oob) == (1, 2)
    assert st.error_word == ora.ERR_DUP_PUT | ora.ERR_OOB_INDEX
    # first write wins: the row of sample 1 is unchanged
    b = d.gather(0, np.array([0, 1, 2, 3], np.int32), want=[rid])
    assert H.bits_equal(b.columns[rid], H.expected_packed(w, rid, [0, 1, 2, 3]))
    # same class, different length -> rejected
    bad_cu = np.array([0, int(w.len_response[0]) + 1], np.int32)
    assert d.put(old, [0], bad_cu, np.zeros(bad_cu[1], np.float32)) == 0
    assert d.stats().n_len_mismatch == 1 and not (d.status()[0] >> old) & 1
    # decreasing cu -> rejected
    assert d.put(rid, [5], np.array([4, 2], np.int32), np.zeros(8, np.int32)) == 0
    assert d.stats().n_bad_length == 1 and d.lengths(2)[5] == -1


def test_arena_full_skips_only_what_does_not_fit():
    cols = [("i32", "response", 0), ("f32", "scalar", 0)]
    d = ora.OracleDock(1, 4, 1, cols, [(3, 3, False)], 8, 24, 1)
    cu = np.array([0, 9, 22, 30, 31], np.int32)        # lengths 9, 13, 8, 1 -> rooms 16, 16, 8, 8
    assert d.put(0, [0, 1, 2, 3], cu, np.arange(31, dtype=np.int32)) == 2
    assert d.lengths(2).tolist() == [9, -1, 8, -1]
    assert d.offsets(2).tolist() == [0, -1, 16, -1]
    assert d.cursors(2).tolist() == [24]
    assert d.stats().n_arena_full == 2 and d.status().tolist() == [1, 0, 1, 0]


def test_output_capacity_truncates_at_group_boundary():
    w = small(schedule="none", G=4, N=2, S=2)
    d = H.make_oracle(w)
    for c in range(len(w.columns)):
        cu, data = w.pack(c, np.arange(w.n, dtype=np.int32))
        d.put(c, np.arange(w.n), cu, data)
    rid = w.column_index("response_ids")
    room = int(w.len_response[:4].sum()) + 1            # two groups fit, the third does not
    b = d.get(0, w.n, capacities={rid: room})
    assert b.indices.tolist() == [0, 1, 2, 3] and b.status == ora.ERR_OUT_TRUNC
    assert H.popcount_words(d.claim_words(0)) == 2     # the skipped groups stay available
    b2 = d.get(0, w.n)
    assert b2.indices.tolist() == [4, 5, 6, 7] and b2.status == 0
    # padded: a row longer than the width stops the batch before its group
    wide = int(w.len_response.max())
    first_long = int(np.argmax(w.len_response == wide))
    b3 = d.get(1, w.n, ora.PADDED, int(w.len_prompt.max()), wide - 1)
    assert b3.n_samples == (first_long // w.N) * w.N and b3.status == ora.ERR_OUT_TRUNC
    # counters: two of the three gets made here were cut; samples and tokens per consumer are
    # those of the batches this test received
    st = d.stats()
    assert st.n_truncated == 2 and st.error_word == ora.ERR_OUT_TRUNC
    tok = lambda idx: int(w.len_prompt[idx].sum() + w.len_response[idx].sum())
    assert st.got_samples[0] == 8 and st.got_tokens[0] == tok(np.arange(8))
    assert st.got_samples[1] == b3.n_samples and st.got_tokens[1] == tok(b3.indices)
    assert st.got_samples[2] == 0 and st.got_tokens[2] == 0


def test_reset_forgets_tables_keeps_payload():
    w = small()
    d = H.make_oracle(w)
    H.replay_oracle(w, d)
    before = d.arena(1, 0).copy()
    d.reset()
    assert not d.status().any() and np.all(d.lengths(2) == -1) and np.all(d.offsets(1) == -1)
    assert not d.cursors(2).any() and H.popcount_words(d.consumed_words(0)) == 0
    assert H.bits_equal(d.arena(1, 0), before)
    assert d.get(0, w.n).n_samples == 0
    # and the dock is usable again, with the same answers
    batches = H.replay_oracle(w, d)
    assert sum(b.n_samples for _, b in batches) == w.n * len(w.consumers)


def test_consumer_masks_are_validated():
    cols = [("i32", "prompt", 0), ("f32", "scalar", 0)]
    with pytest.raises(ValueError):
        ora.OracleDock(2, 2, 1, cols, [(1, 3, False)], 8, 8, 1)     # out not within need
    with pytest.raises(ValueError):
        ora.OracleDock(2, 2, 1, cols, [(1, 1, True)], 8, 8, 1)      # advantage without reward
    with pytest.raises(ValueError):
        ora.OracleDock(3, 2, 2, cols, [(3, 3, False)], 8, 8, 1)     # shards must divide prompts


# ------------------------------------------------- Eq. 1 on the oracle's own output
def test_actor_update_get_moves_eq1_bytes_when_all_lengths_are_maximal():
    """With every prompt at PL and every response at SL, what the actor-update
    consumer receives is Eq. 1's volume: PL + n*SL tokens and M scalars per sample,
    with n = 3 response-length items and M = 3 scalars (index, reward, advantage)."""
    G, N, PL, SL = 4, 4, 24, 56
    w = wl.make_custom("full", G, N, 2, prompt_len=(PL, PL), response=("uniform", SL, SL),
                       vocab=100, micro_batch=G * N, seed=3, schedule="bulk")
    d = H.make_oracle(w)
    (_, b), = [x for x in H.replay_oracle(w, d) if x[0] == 3]
    nbytes = b.indices.nbytes + b.advantages.nbytes + sum(a.nbytes for a in b.columns.values())
    assert nbytes == pytest.approx(ora.cv(G, N, 4, PL, 3, SL, 3) * 1024 ** 3, rel=1e-12)


# ---------------------------------------------------------------- cascade (write-back)
def test_cascade_write_back_round_trip():
    """The whole sample flow on one dock: inference states send a column back for the batch they
    were served.  What the actor update finally receives is pinned without the oracle: the
    test itself remembers which pool row went to which sample, from the batches' index lists
    and the generator's lengths alone."""
    w = small(schedule="cascade", G=12, N=3, S=3, poll_every=4, with_entropy=True, micro_batch=6)
    d = H.make_oracle(w)
    out = H.replay_oracle(w, d)
    # rows each sample was sent, rebuilt from the batches
    sent = {}
    it = iter(out)
    last = {}
    for op in w.ops:
        if op.kind == "get":
            c, b = next(it)
            last[c] = b
        elif op.kind == "put_back":
            b = last[op.consumer]
            lens = w.len_response[b.indices] if b.n_samples else np.zeros(0, np.int32)
            cu = np.concatenate([[0], np.cumsum(lens)])
            for col in op.columns:
                for i, s in enumerate(b.indices):
                    if w.columns[col].cls == wl.SCALAR:
                        sent[(col, int(s))] = w.pool[col][i:i + 1]
                    else:
                        sent[(col, int(s))] = w.pool[col][cu[i]:cu[i + 1]]
    upd = len(w.consumers) - 1
    seen = []
    for c, b in out:
        if c != upd:
            continue
        seen.extend(b.indices.tolist())
        for col, spec in enumerate(w.columns):
            if spec.name in ("prompt_ids", "response_ids"):
                want = H.expected_packed(w, col, b.indices)
            else:
                parts = [sent[(col, int(s))] for s in b.indices]
                want = np.concatenate(parts) if parts else np.zeros(0, w.pool[col].dtype)
            assert H.bits_equal(b.columns[col], want), spec.name
        # advantages from the rewards that were sent back, by numpy
        rcol = w.column_index("reward")
        for g in range(b.n_groups):
            r = np.array([sent[(rcol, int(s))][0] for s in b.indices[g * w.N:(g + 1) * w.N]], dtype=np.float64)
            want = (r - r.mean()) / (r.std() + 1e-6)
            assert np.allclose(b.advantages[g * w.N:(g + 1) * w.N], want.astype(np.float32), rtol=1e-6, atol=1e-7)
    assert sorted(seen) == list(range(w.n))
    for c in range(len(w.consumers)):
        assert sum(b.n_samples for cc, b in out if cc == c) == w.n
    assert d.stats().error_word == 0


# ---------------------------------------------------------------- fused token stream
def _fill_bulk(w, d):
    for c in range(len(w.columns)):
        cu, data = w.pack(c, np.arange(w.n, dtype=np.int32))
        d.put(c, np.arange(w.n), cu, data)


def test_fused_stream_is_prompt_then_response_per_sample():
    """seq equals, sample by sample, the generator's prompt row followed by its response row;
    seq_advantages is 0 over the prompt and the sample's advantage (numpy z-score of its
    group's rewards) over the response; cu_seq indexes both."""
    w = small(schedule="none", G=6, N=3, S=2)
    d = H.make_oracle(w)
    _fill_bulk(w, d)
    pc, rc = w.column_index("prompt_ids"), w.column_index("response_ids")
    upd = len(w.consumers) - 1
    b = d.get(upd, w.n, seq=(pc, rc), seq_adv=True)
    assert b.n_samples == w.n
    sp, sr = w.row_starts(wl.PROMPT), w.row_starts(wl.RESPONSE)
    rew = w.data["reward"].astype(np.float64).reshape(w.G, w.N)
    adv = ((rew - rew.mean(axis=1, keepdims=True)) / (rew.std(axis=1, keepdims=True) + 1e-6)).reshape(-1)
    want_seq, want_adv = [], []
    for s in range(w.n):
        want_seq += [w.data["prompt_ids"][sp[s]:sp[s + 1]], w.data["response_ids"][sr[s]:sr[s + 1]]]
        want_adv += [np.zeros(w.len_prompt[s], np.float32), np.full(w.len_response[s], adv[s], np.float32)]
    assert np.array_equal(b.seq, np.concatenate(want_seq))
    assert np.allclose(b.seq_advantages, np.concatenate(want_adv), rtol=1e-6, atol=1e-7)
    assert np.array_equal(b.cu_seq, np.concatenate([[0], np.cumsum(w.len_prompt + w.len_response)]))
    # the prompt part of the mask is exactly zero, and the response part repeats advantages[i]
    for i in range(w.n):
        a, m, e = b.cu_seq[i], b.cu_seq[i] + w.len_prompt[i], b.cu_seq[i + 1]
        assert not b.seq_advantages[a:m].any()
        assert (b.seq_advantages[m:e] == b.advantages[i]).all()


def test_fused_stream_takes_float_columns_and_respects_capacity():
    """Any prompt/response pair of one element size may be fused; a stream buffer that is too
    small cuts the batch before the first group that does not fit, like any other column."""
    cols = [("f32", "prompt", 0), ("f32", "response", 0), ("bf16", "response", 0), ("f32", "scalar", 0)]
    d = ora.OracleDock(3, 2, 1, cols, [(0xF, 0xF, True)], 256, 256, 3)
    lp, lr = np.array([3, 3, 5, 5, 2, 2]), np.array([4, 1, 0, 7, 6, 6])
    rng = np.random.default_rng(3)
    P, R = rng.random(lp.sum(), dtype=np.float32), rng.random(lr.sum(), dtype=np.float32)
    idx = np.arange(6, dtype=np.int32)
    cup, cur = np.concatenate([[0], np.cumsum(lp)]).astype(np.int32), np.concatenate([[0], np.cumsum(lr)]).astype(np.int32)
    d.put(0, idx, cup, P); d.put(1, idx, cur, R)
    d.put(2, idx, cur, np.zeros(lr.sum(), np.uint16)); d.put(3, idx, None, np.arange(6, dtype=np.float32))
    with pytest.raises(ValueError):
        d.get(0, 6, seq=(0, 2))                       # element sizes differ
    with pytest.raises(ValueError):
        d.get(0, 6, seq=(1, 0))                       # classes swapped
    tot2 = int(lp[:4].sum() + lr[:4].sum())
    b = d.get(0, 6, seq=(0, 1), seq_adv=True, seq_cap=tot2 + 3)     # room for two groups and a bit
    assert b.n_groups == 2 and b.status & ora.ERR_OUT_TRUNC
    want = np.concatenate([np.concatenate([P[cup[i]:cup[i + 1]], R[cur[i]:cur[i + 1]]]) for i in range(4)])
    assert H.bits_equal(b.seq, want)
    b2 = d.get(0, 6, seq=(0, 1), seq_cap=64)          # the group that was cut is still there
    assert b2.n_groups == 1 and list(b2.indices) == [4, 5] and b2.status == 0


def test_cascade_batched_polls_serve_everything_once():
    """The batched form of the cascade (one get call for all worker states, one write-back call
    for all of them per poll) drains like the per-call form: every consumer gets every sample
    exactly once, every column ends up stored for every sample, nothing is flagged."""
    w = small(schedule="cascade_batched", G=12, N=3, S=3, poll_every=4, with_entropy=True, micro_batch=6)
    d = H.make_oracle(w)
    out = H.replay_oracle(w, d)
    for c in range(len(w.consumers)):
        got = np.concatenate([b.indices for cc, b in out if cc == c])
        assert sorted(got.tolist()) == list(range(w.n))
    st = d.stats()
    assert st.error_word == 0
    assert all(st.put_accepted[c] == w.n for c in range(len(w.columns)))
    assert np.all(d.status() == (1 << len(w.columns)) - 1)
