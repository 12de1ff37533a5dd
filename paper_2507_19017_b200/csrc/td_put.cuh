// td_put: reserve rows (alloc), scatter payload into the arenas, publish readiness bits.
// Workflow steps 2 and 3 of "Distributed Transfer Dock Strategy": a worker sends real data to
// the warehouses, then the warehouse state becomes visible to every controller.
#pragma once

#include "td_alloc.cuh"
#include "td_device.cuh"

namespace td {

// Where row i of item `a` goes in its arena if the alloc kernel accepted it, else nullptr; s is
// the row's sample.  Recomputed from the tables, so that a put needs no scratch memory of its own.
__device__ __forceinline__ uint8_t *put_row_dst(const DockView &dv, const PutArgs &a, uint32_t L, uint32_t bit,
                                                uint32_t esz, uint32_t i, int64_t c0, int64_t c1, int32_t &s_out) {
    const int32_t s = a.idx[i];
    if (s < 0 || (uint32_t)s >= dv.n) return nullptr;
    const uint32_t st = dv.status[s];          // three loads side by side
    const int32_t ln = dv.len[L][s];
    const long long off = dv.off[L][s];
    if (st & bit) return nullptr;
    if (c0 < 0 || c1 < c0 || (uint64_t)c1 > a.data_elems) return nullptr;
    if ((int64_t)ln != c1 - c0) return nullptr;
    if (off < 0) return nullptr;
    s_out = s;
    return dv.colbase[a.column] + ((uint64_t)shard_of(dv, (uint32_t)s) * dv.cap[L] + (uint64_t)off) * esz;
}

// What a warp counts while it stores the elements of scalar columns.
struct ScalarCounts {
    uint32_t oob, dup, bad;
};

// Elements [e0, e1) of a scalar item: store, fence, publish.  Returns the number accepted.
// Four elements per lane travel side by side: every step below is a round trip to memory, and a
// warp that took them one after the other would be at it long after the copying warps are done.
__device__ __forceinline__ uint32_t warp_put_scalars(const DockView &dv, const PutArgs &a, uint32_t e0, uint32_t e1,
                                                     uint32_t lane, ScalarCounts &cnt) {
    const uint32_t bit = 1u << a.column, esz = dv.col_esz[a.column];
    uint32_t n_ok = 0;
    for (uint32_t base = e0; base < e1; base += 128) {
        int32_t s[4];
        uint32_t st[4], val[4];
        bool live[4];
        #pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t e = base + lane + 32u * u;
            s[u] = e < e1 ? a.idx[e] : -1;
        }
        #pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t e = base + lane + 32u * u;
            live[u] = false; st[u] = 0; val[u] = 0;
            if (e >= e1) continue;
            if (s[u] < 0 || (uint32_t)s[u] >= dv.n) { ++cnt.oob; continue; }
            if ((uint64_t)e >= a.data_elems) { ++cnt.bad; continue; }
            live[u] = true;
            st[u] = dv.status[s[u]];
            val[u] = esz == 4 ? reinterpret_cast<const uint32_t *>(a.data)[e]
                              : (uint32_t)reinterpret_cast<const uint16_t *>(a.data)[e];
        }
        #pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (!live[u]) continue;
            if (st[u] & bit) { ++cnt.dup; live[u] = false; continue; }
            if (esz == 4) reinterpret_cast<uint32_t *>(dv.colbase[a.column])[s[u]] = val[u];
            else reinterpret_cast<uint16_t *>(dv.colbase[a.column])[s[u]] = (uint16_t)val[u];
        }
        __threadfence();
        #pragma unroll
        for (int u = 0; u < 4; ++u)
            if (live[u]) st[u] = atomicOr(&dv.status[s[u]], bit);
        #pragma unroll
        for (int u = 0; u < 4; ++u) {
            bool ok = false;
            if (live[u]) { if (st[u] & bit) ++cnt.dup; else ok = true; }
            n_ok += __popc(__ballot_sync(kFullMask, ok));
        }
    }
    return n_ok;
}

// Scatter and publish.  The packed sources of the call's items, laid end to end - a ragged row
// charged kRowCost on top of its bytes, an element of a scalar column kPutScalarCost - are cut
// into equal chunks, so that work is balanced over tokens and rows rather than samples; warps
// stride over the chunks (see "Chunked ragged copy" in td_device.cuh).  A row is published by
// the warp that completes it (see warp_copy_chunk), so the call needs no kernel behind this one.
//
// The kernel is launched while the alloc kernel of its call is still running.  With a ready word
// (batch.ready) it does not sit out that kernel's whole run: as soon as the alloc kernel has
// seen everything before the call finish, which it says by storing the call's number there, the
// inputs of the call are safe to read, and this kernel sizes its chunks and brings the index,
// cu and table lines and the first source bytes of each warp's first chunk towards the SM; only
// then does it wait for the alloc kernel itself, whose tables say where the rows go.
constexpr uint32_t kPutScalarCost = 256;       // what an element of a scalar column weighs in the chunked space
static_assert(kPutScalarCost % 16 == 0, "an item's extent stays a multiple of 16");

__global__ void __launch_bounds__(kCopyThreads, kCopyBlocksPerSM)
put_scatter_kernel(const DockView dv, const PutBatch batch) {
    __shared__ uint64_t item_end[kMaxPutItems];       // inclusive prefix of the items' extents (16-byte padded)
    __shared__ uint64_t item_bytes[kMaxPutItems];     // extent of each item (0: nothing to do)
    __shared__ uint32_t item_rows[kMaxPutItems];      // entries of each item
    extern __shared__ __align__(128) uint8_t scatter_smem[];
    const uint32_t tid = threadIdx.x, lane = tid & 31;
    WarpPipe pipe;                                                           // [warps][kPipeSmemPerWarp]
    pipe.init(scatter_smem + (size_t)(tid >> 5) * kPipeSmemPerWarp, lane, dv.spin_limit);
    // Inputs complete?  The alloc kernel says so ahead of its own work; if the word does not show
    // up within the limit, the wait for that kernel's end says the same, only later.
    __shared__ uint32_t s_gave_up;
    __shared__ uint32_t item_base[kMaxPutItems];      // entries of the same class's leader items ahead of the item's leader
    __shared__ uint32_t class_total[3];               // entries of a class's leader items
    bool waited = true;
    if (batch.ready) {
        if (tid == 0) {
            uint32_t polls = 0;
            while (ld_acquire_u64(batch.ready) != (batch.seq << 2) + 2u && ++polls < 4096u) __nanosleep(64);
            s_gave_up = polls >= 4096u;
        }
        __syncthreads();
        waited = s_gave_up != 0;
    }
    if (waited) griddep_wait();                        // the alloc kernel's tables are complete

    if (tid < batch.n_items) {                         // one thread per item: the totals load side by side
        const PutArgs &a = batch.item[tid];
        const uint32_t k = item_k(a);
        uint64_t bytes = 0;
        if (k) {
            if (dv.col_cls[a.column] == TD_SCALAR) {
                bytes = (uint64_t)k * kPutScalarCost;
            } else {
                const int64_t tot = a.cu[k];
                if (tot >= 0 && (uint64_t)tot <= a.data_elems)
                    bytes = (uint64_t)tot * dv.col_esz[a.column] + (uint64_t)k * kRowCost;
            }
        }
        item_bytes[tid] = bytes;
        item_rows[tid] = k;
    }
    __syncthreads();
    if (tid == 0) {
        uint64_t acc = 0;
        uint32_t seen[3] = {0, 0, 0};
        for (uint32_t it = 0; it < batch.n_items; ++it) {
            acc += (item_bytes[it] + 15) & ~uint64_t(15);
            item_end[it] = acc;
            // where the alloc kernel's count of entries stands when it reaches this item's rows:
            // a follower's rows are settled with its leader's
            const uint32_t L = dv.col_cls[batch.item[it].column];
            if (batch.follow[it]) item_base[it] = item_base[batch.follow[it] - 1u];
            else { item_base[it] = seen[L]; seen[L] += item_rows[it]; }
        }
        class_total[0] = 0; class_total[1] = seen[1]; class_total[2] = seen[2];
    }
    __syncthreads();
    const uint64_t n_warps = (uint64_t)gridDim.x * kCopyWarps;
    const uint64_t total = item_end[batch.n_items - 1];
    // With plenty to do (a full-size chunk and more per warp) and a counter to draw from, the
    // chunks after a warp's first are handed out one by one: equal bytes are not equal time, and
    // some SMs get through theirs sooner than others.  Otherwise every warp takes a fixed share.
    unsigned long long *work_counter = total >= n_warps * (uint64_t)kChunkTargetBytes ? batch.work_counter : nullptr;
    const ChunkPlan plan = work_counter ? plan_chunks_dynamic(total, n_warps) : plan_chunks(total, n_warps);
    unsigned long long ch = (uint64_t)blockIdx.x * kCopyWarps + (tid >> 5);

    if (!waited) {
        // Ahead of the alloc kernel's end: what the warp's first chunk will ask for, asked for now.
        if (ch < plan.n_chunks) {
            const uint64_t g0 = ch * plan.chunk_bytes;
            uint32_t it = 0;
            while (item_end[it] <= g0) ++it;
            const PutArgs &a = batch.item[it];
            const uint32_t L = dv.col_cls[a.column], esz = dv.col_esz[a.column];
            const uint64_t b0 = g0 - (it ? item_end[it - 1] : 0);
            if (L != TD_SCALAR && item_rows[it] && b0 < item_bytes[it]) {
                const uint32_t r0 = warp_find_row(a.cu, item_rows[it], (int64_t)b0, esz, kRowCost, lane, a.idx);
                const uint32_t i = r0 + lane;
                if (i < item_rows[it]) {
                    const int64_t c0 = __ldg(a.cu + i);
                    const int32_t s = a.idx[i];
                    if (s >= 0 && (uint32_t)s < dv.n) {
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(dv.status + s));
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(dv.len[L] + s));
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(dv.off[L] + s));
                    }
                    // the head of the row (the first row: from where the chunk starts in it)
                    if (c0 >= 0 && (uint64_t)c0 < a.data_elems) {
                        const uint64_t row0 = (uint64_t)c0 * esz + (uint64_t)i * kRowCost + kRowCost;
                        const uint64_t skip = lane == 0 && b0 > row0 ? b0 - row0 : 0;
                        const uint8_t *p = a.data + (uint64_t)c0 * esz + skip;
                        const uint8_t *end = a.data + a.data_elems * esz;
                        #pragma unroll
                        for (int q = 0; q < 4; ++q)
                            if (p + 128 * q < end) asm volatile("prefetch.global.L2 [%0];" ::"l"(p + 128 * q));
                    }
                }
            }
        }
        // with a count of the entries allocated so far, rows are waited for one chunk at a time
        if (!batch.progress || (*dv.errword & kErrIrregularCu)) { griddep_wait(); waited = true; }
    }
    // Nothing behind this kernel needs it to have finished before it starts setting itself up.
    griddep_launch_dependents();
    // Rows [0, need) of the item being copied have their places once the alloc kernel's count for
    // the item's class has reached item_base + need.  One lane polls; when the count does not get
    // there within the limit, the wait for that kernel's end settles it, as it does once for all
    // when the call has no such count.
    bool done_prompt = waited, done_response = waited;       // the class's count has reached its total
    uint32_t cur_item = 0, cur_class = 0;
    auto await = [&](uint32_t need_rows) {
        if (cur_class == TD_PROMPT ? done_prompt : done_response) return;
        const uint32_t need = item_base[cur_item] + need_rows;
        unsigned long long v = 0;
        if (lane == 0) {
            uint32_t polls = 0;
            for (;;) {
                v = ld_acquire_u64(&batch.progress[cur_class - 1u]);
                if (((uint32_t)(v >> 32) == (uint32_t)batch.seq && (uint32_t)v >= need) || ++polls >= 16384u) break;
                __nanosleep(100);
            }
        }
        v = shfl_u64(v, 0);
        if ((uint32_t)(v >> 32) != (uint32_t)batch.seq || (uint32_t)v < need) {
            griddep_wait();
            done_prompt = done_response = true;
        } else if ((uint32_t)v >= class_total[cur_class]) {
            if (cur_class == TD_PROMPT) done_prompt = true; else done_response = true;
        }
        __syncwarp();
    };

    ScalarCounts cnt{0, 0, 0};
    PublishQueue queue;
    publish_queue_init(queue);
    // A cu array that is not a non-decreasing sequence inside its data (the alloc kernel of this
    // call, or of an earlier one since the last reset, met one) gives rows no searchable position:
    // the warps then take the rows of every item one by one, each row checked for itself, so that
    // exactly the rows the alloc kernel accepted are copied and published.
    if (*dv.errword & kErrIrregularCu) {
        for (uint32_t it = 0; it < batch.n_items; ++it) {
            const PutArgs &a = batch.item[it];
            const uint32_t L = dv.col_cls[a.column], esz = dv.col_esz[a.column], bit = 1u << a.column;
            uint32_t n_ok = 0;
            const uint64_t w0 = (uint64_t)blockIdx.x * kCopyWarps + (tid >> 5);
            if (L == TD_SCALAR) {
                for (uint64_t e = w0 * 128; e < item_rows[it]; e += n_warps * 128)
                    n_ok += warp_put_scalars(dv, a, (uint32_t)e, (uint32_t)min(e + 128, (uint64_t)item_rows[it]), lane, cnt);
            } else {
                const uint8_t *lo = a.data, *hi = a.data + a.data_elems * esz;
                for (uint64_t i = w0; i < item_rows[it]; i += n_warps) {
                    const int64_t c0 = a.cu[i], c1 = a.cu[i + 1];
                    int32_t s = -1;
                    uint8_t *dst = put_row_dst(dv, a, L, bit, esz, (uint32_t)i, c0, c1, s);
                    if (!dst) continue;
                    const uint8_t *src = a.data + (uint64_t)c0 * esz;
                    for (uint64_t left = (uint64_t)(c1 - c0) * esz; left; ) {
                        const uint32_t m = (uint32_t)min(left, (uint64_t)1 << 30);
                        pipe.push<true>(dst, src, m, lane, lo, hi);
                        dst += m; src += m; left -= m;
                    }
                    pipe.drain_all(lane);
                    __threadfence();
                    __syncwarp();
                    if (lane == 0 && !(atomicOr(&dv.status[s], bit) & bit)) ++n_ok;
                }
                n_ok = __reduce_add_sync(kFullMask, n_ok);
            }
            if (lane == 0 && n_ok) atomicAdd(&dv.counters[CNT_PUT_ACCEPTED + a.column], (unsigned long long)n_ok);
        }
    } else {
        while (ch < plan.n_chunks) {
            unsigned long long next = ch + n_warps;
            if (work_counter) {
                if (lane == 0) next = n_warps + atomicAdd(work_counter, 1ull);    // in flight while this chunk is copied
                // (handed to the other lanes at the end of the loop body)
            }
            uint64_t g0 = ch * plan.chunk_bytes;
            const uint64_t g1 = min(g0 + plan.chunk_bytes, total);
            uint32_t it = 0;
            while (item_end[it] <= g0) ++it;
            for (; g0 < g1; ++it) {
                const uint64_t start = it ? item_end[it - 1] : 0;
                const PutArgs &a = batch.item[it];
                const uint32_t L = dv.col_cls[a.column];
                const uint32_t esz = dv.col_esz[a.column];
                const uint32_t bit = 1u << a.column;
                const uint64_t b0 = g0 - start;
                g0 = min(g1, item_end[it]);
                if (item_rows[it] == 0) continue;
                const uint64_t b1 = min(g0 - start, item_bytes[it]);
                if (b1 <= b0) continue;
                if (L == TD_SCALAR) {
                    // element e belongs to the chunk that holds byte e * kPutScalarCost of the item
                    const uint32_t e0 = (uint32_t)((b0 + kPutScalarCost - 1) / kPutScalarCost);
                    const uint32_t e1 = (uint32_t)min((b1 + kPutScalarCost - 1) / kPutScalarCost, (uint64_t)item_rows[it]);
                    const uint32_t n_ok = warp_put_scalars(dv, a, e0, e1, lane, cnt);
                    if (lane == 0 && n_ok) atomicAdd(&dv.counters[CNT_PUT_ACCEPTED + a.column], (unsigned long long)n_ok);
                } else {
                    cur_item = it; cur_class = L;
                    warp_copy_chunk<false, true>(
                        a.cu, item_rows[it], b0, b1, const_cast<uint8_t *>(a.data), esz, lane,
                        a.data, a.data + a.data_elems * esz, pipe, a.idx,
                        [&](uint32_t i, int64_t c0, int64_t c1, int32_t &s) -> uint8_t * {
                            return put_row_dst(dv, a, L, bit, esz, i, c0, c1, s);     // live if the alloc kernel accepted it
                        },
                        nullptr, false, &dv, &queue, a.column, await);
                }
            }
            ch = work_counter ? shfl_u64(next, 0) : next;
        }
    }
    publish_queue_flush(dv, queue, pipe, lane);
    if (pipe.finish(lane) && lane == 0) flag_error(dv, TD_ERR_COPY_TIMEOUT, CNT_TIMEOUT);
    // This kernel's end must imply the alloc kernel's (whatever follows in the stream waits for
    // this one only); by now that kernel is long done.
    if (!waited) griddep_wait();
    cnt.oob = __reduce_add_sync(kFullMask, cnt.oob);
    cnt.dup = __reduce_add_sync(kFullMask, cnt.dup);
    cnt.bad = __reduce_add_sync(kFullMask, cnt.bad);
    if (lane == 0) {
        if (cnt.oob) flag_error(dv, TD_ERR_OOB_INDEX, CNT_OOB, cnt.oob);
        if (cnt.dup) flag_error(dv, TD_ERR_DUP_PUT, CNT_DUP, cnt.dup);
        if (cnt.bad) flag_error(dv, TD_ERR_BAD_LENGTH, CNT_BADLEN, cnt.bad);
    }
}

// Publish of a call that holds scalar columns only (a reward, say): there is nothing to scatter,
// one thread stores its element and sets the sample's bit behind a fence.
__global__ void __launch_bounds__(256)
put_publish_kernel(const DockView dv, const PutBatch batch) {
    // the kernel ahead may be the one that produces this call's index array: everything waits
    griddep_wait();
    griddep_launch_dependents();
    uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t it = 0;
    for (; it < batch.n_items; ++it) {                 // grid slots are laid out by the items' largest counts
        if (i < batch.item[it].k) break;
        i -= batch.item[it].k;
    }
    if (it < batch.n_items && i >= item_k(batch.item[it])) it = batch.n_items;
    uint32_t ok = 0, n_oob = 0, n_dup = 0, n_bad = 0, column = 0;
    if (it < batch.n_items) {
        const PutArgs &a = batch.item[it];
        column = a.column;
        const uint32_t bit = 1u << column;
        const int32_t s = a.idx[i];
        if (s < 0 || (uint32_t)s >= dv.n) ++n_oob;
        else if ((uint64_t)i >= a.data_elems) ++n_bad;
        else if (dv.status[s] & bit) ++n_dup;
        else {
            if (dv.col_esz[column] == 4) reinterpret_cast<uint32_t *>(dv.colbase[column])[s] = reinterpret_cast<const uint32_t *>(a.data)[i];
            else reinterpret_cast<uint16_t *>(dv.colbase[column])[s] = reinterpret_cast<const uint16_t *>(a.data)[i];
            __threadfence();
            if (atomicOr(&dv.status[s], bit) & bit) ++n_dup; else ok = 1;
        }
    }
    // a warp may straddle two items: count per column with a match on the column number
    const uint32_t peers = __match_any_sync(kFullMask, column);
    const uint32_t okc = __popc(__ballot_sync(kFullMask, ok) & peers);
    if (okc && (threadIdx.x & 31) == (uint32_t)__ffs(peers) - 1u)
        atomicAdd(&dv.counters[CNT_PUT_ACCEPTED + column], (unsigned long long)okc);
    n_oob = __reduce_add_sync(kFullMask, n_oob);
    n_dup = __reduce_add_sync(kFullMask, n_dup);
    n_bad = __reduce_add_sync(kFullMask, n_bad);
    if ((threadIdx.x & 31) == 0) {
        if (n_oob) flag_error(dv, TD_ERR_OOB_INDEX, CNT_OOB, n_oob);
        if (n_dup) flag_error(dv, TD_ERR_DUP_PUT, CNT_DUP, n_dup);
        if (n_bad) flag_error(dv, TD_ERR_BAD_LENGTH, CNT_BADLEN, n_bad);
    }
}

}  // namespace td
