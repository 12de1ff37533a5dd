// td_put: reserve rows (alloc), scatter payload into the arenas, publish readiness bits.
// Workflow steps 2 and 3 of "Distributed Transfer Dock Strategy": a worker sends real data to
// the warehouses, then the warehouse state becomes visible to every controller.
#pragma once

#include "td_alloc.cuh"
#include "td_device.cuh"

namespace td {

// Is entry i of this item a row that the alloc kernel accepted?  Recomputed from the tables by
// the scatter and publish kernels, so that a put needs no scratch memory of its own.
__device__ __forceinline__ bool put_entry_live(const DockView &dv, const PutArgs &a, uint32_t i,
                                               uint32_t L, uint32_t bit, int32_t &s_out,
                                               int64_t &len_out, long long &off_out) {
    // two rounds of loads: the entry, then the three table words behind its index
    const int32_t s = a.idx[i];
    const int64_t c0 = a.cu[i], c1 = a.cu[i + 1];
    if (s < 0 || (uint32_t)s >= dv.n) return false;
    const uint32_t st = dv.status[s];
    const int32_t ln = dv.len[L][s];
    const long long off = dv.off[L][s];
    if (st & bit) return false;
    const int64_t l = c1 - c0;
    if (l < 0 || c0 < 0 || (uint64_t)c1 > a.data_elems) return false;
    if ((int64_t)ln != l) return false;
    if (off < 0) return false;
    s_out = s; len_out = l; off_out = off;
    return true;
}

// Where row i of item `a` goes in its arena if the alloc kernel accepted it, else nullptr.
__device__ __forceinline__ uint8_t *put_row_dst(const DockView &dv, const PutArgs &a, uint32_t L, uint32_t bit,
                                                uint32_t esz, uint32_t i, int64_t c0, int64_t c1) {
    const int32_t s = a.idx[i];
    if (s < 0 || (uint32_t)s >= dv.n) return nullptr;
    const uint32_t st = dv.status[s];          // three loads side by side
    const int32_t ln = dv.len[L][s];
    const long long off = dv.off[L][s];
    if (st & bit) return nullptr;
    if (c0 < 0 || c1 < c0 || (uint64_t)c1 > a.data_elems) return nullptr;
    if ((int64_t)ln != c1 - c0) return nullptr;
    if (off < 0) return nullptr;
    return dv.colbase[a.column] + ((uint64_t)shard_of(dv, (uint32_t)s) * dv.cap[L] + (uint64_t)off) * esz;
}

// Scatter.  The packed sources of the call's ragged items, laid end to end with every row
// charged kRowCost on top of its bytes, are cut into equal chunks, so that work is balanced
// over tokens and rows rather than samples; warps stride over the chunks (see "Chunked ragged
// copy" in td_device.cuh).
__global__ void __launch_bounds__(kCopyThreads, kCopyBlocksPerSM)
put_scatter_kernel(const DockView dv, const PutBatch batch) {
    __shared__ uint64_t item_end[kMaxPutItems];       // inclusive prefix of the items' extents (16-byte padded)
    __shared__ uint64_t item_bytes[kMaxPutItems];     // extent of each ragged item: bytes + rows * kRowCost (0: nothing to copy)
    __shared__ uint32_t item_rows[kMaxPutItems];      // entries of each item
    extern __shared__ __align__(128) uint8_t scatter_smem[];
    const uint32_t tid = threadIdx.x, lane = tid & 31;
    WarpPipe pipe;                                                           // [warps][kPipeSmemPerWarp]
    pipe.init(scatter_smem + (size_t)(tid >> 5) * kPipeSmemPerWarp, lane, dv.spin_limit);
    griddep_wait();                                    // the alloc kernel's tables are complete
    // Only now may the publish kernel be brought on: it reads the call's arrays and the tables
    // ahead of its own wait, which is safe once everything before this kernel has finished.
    griddep_launch_dependents();

    if (tid < batch.n_items) {                         // one thread per item: the totals load side by side
        const PutArgs &a = batch.item[tid];
        const uint32_t k = item_k(a);
        uint64_t bytes = 0;
        if (dv.col_cls[a.column] != TD_SCALAR && k) {
            const int64_t tot = a.cu[k];
            if (tot > 0 && (uint64_t)tot <= a.data_elems)
                bytes = (uint64_t)tot * dv.col_esz[a.column] + (uint64_t)k * kRowCost;
        }
        item_bytes[tid] = bytes;
        item_rows[tid] = k;
    }
    __syncthreads();
    if (tid == 0) {
        uint64_t acc = 0;
        for (uint32_t it = 0; it < batch.n_items; ++it) {
            acc += (item_bytes[it] + 15) & ~uint64_t(15);
            item_end[it] = acc;
        }
    }
    __syncthreads();
    const uint64_t n_warps = (uint64_t)gridDim.x * kCopyWarps;
    // A cu array that is not a non-decreasing sequence inside its data (the alloc kernel of this
    // call, or of an earlier one since the last reset, met one) gives rows no searchable position:
    // the warps then take the rows of every item one by one, each row checked for itself, so that
    // exactly the rows the alloc kernel accepted are copied, as the publish kernel assumes.
    if (*dv.errword & kErrIrregularCu) {
        for (uint32_t it = 0; it < batch.n_items; ++it) {
            const PutArgs &a = batch.item[it];
            const uint32_t L = dv.col_cls[a.column], esz = dv.col_esz[a.column];
            if (L == TD_SCALAR) continue;
            const uint8_t *lo = a.data, *hi = a.data + a.data_elems * esz;
            for (uint64_t i = (uint64_t)blockIdx.x * kCopyWarps + (tid >> 5); i < item_rows[it]; i += n_warps) {
                const int64_t c0 = a.cu[i], c1 = a.cu[i + 1];
                uint8_t *dst = put_row_dst(dv, a, L, 1u << a.column, esz, (uint32_t)i, c0, c1);
                if (!dst) continue;
                const uint8_t *src = a.data + (uint64_t)c0 * esz;
                for (uint64_t left = (uint64_t)(c1 - c0) * esz; left; ) {
                    const uint32_t m = (uint32_t)min(left, (uint64_t)1 << 30);
                    pipe.push<true>(dst, src, m, lane, lo, hi);
                    dst += m; src += m; left -= m;
                }
            }
        }
        if (pipe.finish(lane) && lane == 0) flag_error(dv, TD_ERR_COPY_TIMEOUT, CNT_TIMEOUT);
        return;
    }
    // With plenty to do (a full-size chunk and more per warp) and a counter to draw from, the
    // chunks after a warp's first are handed out one by one: equal bytes are not equal time, and
    // some SMs get through theirs sooner than others.  Otherwise every warp takes a fixed share.
    const uint64_t total = item_end[batch.n_items - 1];
    unsigned long long *work_counter = total >= n_warps * (uint64_t)kChunkTargetBytes ? batch.work_counter : nullptr;
    const ChunkPlan plan = work_counter ? plan_chunks_dynamic(total, n_warps) : plan_chunks(total, n_warps);
    unsigned long long ch = (uint64_t)blockIdx.x * kCopyWarps + (tid >> 5);

    while (ch < plan.n_chunks) {
        unsigned long long next = ch + n_warps;
        if (work_counter) {
            if (lane == 0) next = n_warps + atomicAdd(work_counter, 1ull);    // in flight while this chunk is copied
            // (handed to the other lanes at the end of the loop body)
        }
        uint64_t g0 = ch * plan.chunk_bytes;
        const uint64_t g1 = min(g0 + plan.chunk_bytes, item_end[batch.n_items - 1]);
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
            if (L == TD_SCALAR || item_rows[it] == 0) continue;
            const uint64_t b1 = min(g0 - start, item_bytes[it]);
            if (b1 <= b0) continue;
            warp_copy_chunk<false>(a.cu, item_rows[it], b0, b1, const_cast<uint8_t *>(a.data), esz, lane,
                                   a.data, a.data + a.data_elems * esz, pipe, a.idx,
                                   [&](uint32_t i, int64_t c0, int64_t c1) -> uint8_t * {
                                       return put_row_dst(dv, a, L, bit, esz, i, c0, c1);   // live if the alloc kernel accepted it
                                   });
        }
        ch = work_counter ? shfl_u64(next, 0) : next;
    }
    if (pipe.finish(lane) && lane == 0) flag_error(dv, TD_ERR_COPY_TIMEOUT, CNT_TIMEOUT);
}

// Publish.  Runs after the scatter kernel has finished, so every payload byte of the call is
// globally visible before a readiness bit is; the fence orders the bit behind them for readers
// that acquire it.  A scalar item needs no scatter: its element is stored here, then published.
__global__ void __launch_bounds__(256)
put_publish_kernel(const DockView dv, const PutBatch batch, const uint32_t behind_scatter) {
    // behind_scatter: this launch follows the call's scatter kernel, which let it start only
    // after the alloc kernel had finished: the entry and its table words can be fetched while the
    // scatter is still copying, and only the readiness bit has to wait for it.  Otherwise (a
    // call of scalar columns only) the kernel ahead may be the one that produces this call's
    // index array, and everything waits.
    if (!behind_scatter) griddep_wait();
    uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t it = 0;
    for (; it < batch.n_items; ++it) {                 // grid slots are laid out by the items' largest counts
        if (i < batch.item[it].k) break;
        i -= batch.item[it].k;
    }
    if (it < batch.n_items && i >= item_k(batch.item[it])) it = batch.n_items;
    uint32_t ok = 0, n_oob = 0, n_dup = 0, n_bad = 0, column = 0;
    int32_t s = -1;                                    // sample whose bit this thread sets, if any
    uint32_t bit = 0, value = 0;
    bool store_scalar = false;
    if (it < batch.n_items) {
        const PutArgs &a = batch.item[it];
        column = a.column;
        const uint32_t L = dv.col_cls[column];
        bit = 1u << column;
        if (L != TD_SCALAR) {
            int32_t ss; int64_t l; long long off;
            if (put_entry_live(dv, a, i, L, bit, ss, l, off)) s = ss;
        } else {
            const int32_t ss = a.idx[i];
            if (ss < 0 || (uint32_t)ss >= dv.n) ++n_oob;
            else if ((uint64_t)i >= a.data_elems) ++n_bad;
            else if (dv.status[ss] & bit) ++n_dup;
            else {
                value = dv.col_esz[column] == 4 ? reinterpret_cast<const uint32_t *>(a.data)[i]
                                                : (uint32_t)reinterpret_cast<const uint16_t *>(a.data)[i];
                store_scalar = true;
                s = ss;
            }
        }
    }
    if (behind_scatter) griddep_wait();                // every payload byte of the call is in place
    if (s >= 0) {
        if (store_scalar) {
            if (dv.col_esz[column] == 4) reinterpret_cast<uint32_t *>(dv.colbase[column])[s] = value;
            else reinterpret_cast<uint16_t *>(dv.colbase[column])[s] = (uint16_t)value;
        }
        __threadfence();
        const uint32_t old = atomicOr(&dv.status[s], bit);
        if (old & bit) { if (store_scalar) ++n_dup; } else ok = 1;
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
