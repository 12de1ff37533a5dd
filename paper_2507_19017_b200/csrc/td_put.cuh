// td_put: reserve rows (alloc), scatter payload into the arenas, publish readiness bits.
// Workflow steps 2 and 3 of "Distributed Transfer Dock Strategy": a worker sends real data to
// the warehouses, then the warehouse state becomes visible to every controller.
#pragma once

#include "td_device.cuh"

namespace td {

constexpr int kAllocThreads = 1024;
constexpr int kAllocWarps = kAllocThreads / 32;
constexpr int kMaxPutItems = 8;                // columns one put launch can carry
constexpr uint32_t kNotAllocating = 0xffffffffu;

struct PutArgs {
    uint32_t column, k;
    const int32_t *idx;
    const int32_t *cu;
    const uint8_t *data;
    uint64_t data_elems;
};
struct PutBatch {                              // the columns of one call, in call order
    uint32_t n_items;
    uint32_t pad;
    PutArgs item[kMaxPutItems];
};

// Is entry i of this item a row that the alloc kernel accepted?  Recomputed from the tables by
// the scatter and publish kernels, so that a put needs no scratch memory of its own.
__device__ __forceinline__ bool put_entry_live(const DockView &dv, const PutArgs &a, uint32_t i,
                                               uint32_t L, uint32_t bit, int32_t &s_out,
                                               int64_t &len_out, long long &off_out) {
    const int32_t s = a.idx[i];
    if (s < 0 || (uint32_t)s >= dv.n) return false;
    if (dv.status[s] & bit) return false;
    const int64_t c0 = a.cu[i], c1 = a.cu[i + 1];
    const int64_t l = c1 - c0;
    if (l < 0 || c0 < 0 || (uint64_t)c1 > a.data_elems) return false;
    if ((int64_t)dv.len[L][s] != l) return false;
    const long long off = dv.off[L][s];
    if (off < 0) return false;
    s_out = s; len_out = l; off_out = off;
    return true;
}

static inline size_t put_alloc_smem_bytes(uint32_t S) {
    return (size_t)(kAllocWarps + 2) * S * sizeof(unsigned long long);
}

// Alloc.  One CTA walks the ragged items of the call one after the other, each in rounds of
// kAllocThreads entries in call order.  Per round: validate, decide who reserves a row (first
// arrival of the length class, settled by a CAS on len), then an ordered per-shard exclusive
// scan of the row sizes gives every new row the offset a sequential walk would have given it.
// A round that would overflow a shard is replayed by one thread, entry by entry, so that only
// the rows without room are refused.
__global__ void __launch_bounds__(kAllocThreads)
put_alloc_kernel(const DockView dv, const PutBatch batch) {
    extern __shared__ unsigned long long smem_u64[];
    const uint32_t S = dv.S;
    unsigned long long *tot = smem_u64;                            // [kAllocWarps][S]
    unsigned long long *s_total = tot + (size_t)kAllocWarps * S;   // [S] row space asked per shard
    unsigned long long *s_start = s_total + S;                     // [S] where the round's space begins
    __shared__ int32_t e_s[kAllocThreads];
    __shared__ uint32_t e_room[kAllocThreads];
    __shared__ uint32_t s_overflow;

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t n_oob = 0, n_dup = 0, n_bad = 0, n_mis = 0, n_full = 0;

    for (uint32_t it = 0; it < batch.n_items; ++it) {
        const PutArgs &a = batch.item[it];
        const uint32_t L = dv.col_cls[a.column];
        if (L == TD_SCALAR) continue;
        const uint32_t bit = 1u << a.column;
        const uint64_t cap = dv.cap[L];
        for (uint32_t base = 0; base < a.k; base += kAllocThreads) {
            for (uint32_t j = tid; j < kAllocWarps * S; j += kAllocThreads) tot[j] = 0;
            if (tid == 0) s_overflow = 0;
            const uint32_t i = base + tid;
            bool alloc = false;
            int32_t s = -1;
            uint32_t room = 0, sh = 0;
            if (i < a.k) {
                s = a.idx[i];
                if (s < 0 || (uint32_t)s >= dv.n) { ++n_oob; }
                else if (dv.status[s] & bit) { ++n_dup; }
                else {
                    const int64_t c0 = a.cu[i], c1 = a.cu[i + 1];
                    const int64_t l = c1 - c0;
                    if (l < 0 || c0 < 0 || (uint64_t)c1 > a.data_elems) { ++n_bad; }
                    else {
                        const int32_t old = atomicCAS(&dv.len[L][s], -1, (int32_t)l);
                        if (old == -1) {
                            alloc = true;
                            room = (uint32_t)align_row((uint64_t)l);
                            sh = shard_of(dv, (uint32_t)s);
                        } else if (old != (int32_t)l) { ++n_mis; }
                    }
                }
            }
            e_s[tid] = s;
            e_room[tid] = alloc ? room : kNotAllocating;
            // ordered exclusive prefix per shard inside the warp
            const uint32_t key = alloc ? sh : kNotAllocating;
            unsigned long long pre = 0, wsum = 0;
            bool leader = alloc;
            #pragma unroll 8
            for (uint32_t j = 0; j < 32; ++j) {
                const uint32_t kj = __shfl_sync(kFullMask, key, j);
                const uint32_t rj = __shfl_sync(kFullMask, room, j);
                if (alloc && kj == key) {
                    wsum += rj;
                    if (j < lane) { pre += rj; leader = false; }
                }
            }
            __syncthreads();                                   // tot zeroed, e_* written
            if (leader) tot[warp * S + sh] = wsum;
            __syncthreads();
            // per shard: exclusive scan of the warps' sums in warp order, then reserve
            for (uint32_t key2 = warp; key2 < S; key2 += kAllocWarps) {
                const unsigned long long v = tot[lane * S + key2];
                unsigned long long inc = v;
                #pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const unsigned long long t = __shfl_up_sync(kFullMask, inc, d);
                    if ((int)lane >= d) inc += t;
                }
                tot[lane * S + key2] = inc - v;
                if (lane == 31) {
                    s_total[key2] = inc;
                    // rows of length zero still get a place: the cursor as it stands
                    const unsigned long long start = atomicAdd(&dv.cursor[L][key2], inc);
                    if (start + inc > cap) s_overflow = 1;
                    s_start[key2] = start;
                }
            }
            __syncthreads();
            if (!s_overflow) {
                if (alloc) dv.off[L][s] = (long long)(s_start[sh] + tot[warp * S + sh] + pre);
            } else {
                // hand the round's reservations back, then replay the round in call order
                for (uint32_t key2 = tid; key2 < S; key2 += kAllocThreads)
                    atomicAdd(&dv.cursor[L][key2], 0ull - s_total[key2]);
                __syncthreads();
                if (tid == 0) {
                    for (uint32_t t = 0; t < kAllocThreads; ++t) {
                        const uint32_t r = e_room[t];
                        if (r == kNotAllocating) continue;
                        const int32_t ss = e_s[t];
                        const uint32_t key2 = shard_of(dv, (uint32_t)ss);
                        const unsigned long long start = atomicAdd(&dv.cursor[L][key2], (unsigned long long)r);
                        if (start + r > cap) {
                            atomicAdd(&dv.cursor[L][key2], 0ull - (unsigned long long)r);
                            atomicExch(&dv.len[L][ss], -1);
                            ++n_full;
                        } else {
                            dv.off[L][ss] = (long long)start;
                        }
                    }
                }
            }
            __syncthreads();
        }
        __threadfence_block();
    }
    n_oob = __reduce_add_sync(kFullMask, n_oob);
    n_dup = __reduce_add_sync(kFullMask, n_dup);
    n_bad = __reduce_add_sync(kFullMask, n_bad);
    n_mis = __reduce_add_sync(kFullMask, n_mis);
    n_full = __reduce_add_sync(kFullMask, n_full);
    if (lane == 0) {
        if (n_oob) flag_error(dv, TD_ERR_OOB_INDEX, CNT_OOB, n_oob);
        if (n_dup) flag_error(dv, TD_ERR_DUP_PUT, CNT_DUP, n_dup);
        if (n_bad) flag_error(dv, TD_ERR_BAD_LENGTH, CNT_BADLEN, n_bad);
        if (n_mis) flag_error(dv, TD_ERR_LEN_MISMATCH, CNT_MISMATCH, n_mis);
        if (n_full) flag_error(dv, TD_ERR_ARENA_FULL, CNT_FULL, n_full);
    }
}

// Scatter.  The packed sources of the call's ragged items, laid end to end, are cut into equal
// chunks, so that work is balanced over tokens rather than samples; warps stride over the
// chunks (see "Chunked ragged copy" in td_device.cuh).
__global__ void __launch_bounds__(kCopyThreads, kCopyBlocksPerSM)
put_scatter_kernel(const DockView dv, const PutBatch batch) {
    __shared__ uint64_t item_end[kMaxPutItems];       // inclusive prefix of bytes (16-byte padded) per item
    extern __shared__ __align__(128) uint8_t scatter_smem[];
    uint8_t *stages = scatter_smem;                                          // [warps][stages][kStageBytes]
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(stages + kCopyWarps * kStages * kStageBytes);
    const uint32_t tid = threadIdx.x, lane = tid & 31;
    WarpPipe pipe;
    pipe.init(stages + (size_t)(tid >> 5) * kStages * kStageBytes, bars + (tid >> 5) * kStages, lane, dv.spin_limit);

    if (tid == 0) {
        uint64_t acc = 0;
        for (uint32_t it = 0; it < batch.n_items; ++it) {
            const PutArgs &a = batch.item[it];
            uint64_t bytes = 0;
            if (dv.col_cls[a.column] != TD_SCALAR && a.k) {
                const int64_t tot = a.cu[a.k];
                if (tot > 0 && (uint64_t)tot <= a.data_elems) bytes = (uint64_t)tot * dv.col_esz[a.column];
            }
            acc += (bytes + 15) & ~uint64_t(15);
            item_end[it] = acc;
        }
    }
    __syncthreads();
    const uint64_t n_warps = (uint64_t)gridDim.x * kCopyWarps;
    const ChunkPlan plan = plan_chunks(item_end[batch.n_items - 1], n_warps);
    const uint64_t warp0 = (uint64_t)blockIdx.x * kCopyWarps + (tid >> 5);

    for (uint64_t ch = warp0; ch < plan.n_chunks; ch += n_warps) {
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
            if (L == TD_SCALAR || a.k == 0) continue;
            const uint64_t total_bytes = (uint64_t)(int64_t)__ldg(a.cu + a.k) * esz;
            const uint64_t b1 = min(g0 - start, total_bytes);
            if (b1 <= b0) continue;
            uint8_t *arena = dv.colbase[a.column];
            const uint64_t cap = dv.cap[L];
            warp_copy_chunk<false>(a.cu, a.k, b0, b1, const_cast<uint8_t *>(a.data), esz, lane,
                                   a.data, a.data + a.data_elems * esz, pipe,
                                   [&](uint32_t i, int64_t c0, int64_t c1) -> uint8_t * {
                                       // the row is live if the alloc kernel accepted it
                                       const int32_t s = a.idx[i];
                                       if (s < 0 || (uint32_t)s >= dv.n) return nullptr;
                                       if (dv.status[s] & bit) return nullptr;
                                       if (c1 < c0 || (uint64_t)c1 > a.data_elems) return nullptr;
                                       if ((int64_t)dv.len[L][s] != c1 - c0) return nullptr;
                                       const long long off = dv.off[L][s];
                                       if (off < 0) return nullptr;
                                       return arena + ((uint64_t)shard_of(dv, (uint32_t)s) * cap + (uint64_t)off) * esz;
                                   });
        }
    }
    if (pipe.finish(lane) && lane == 0) flag_error(dv, TD_ERR_COPY_TIMEOUT, CNT_TIMEOUT);
}

// Publish.  Runs after the scatter kernel has finished, so every payload byte of the call is
// globally visible before a readiness bit is; the fence orders the bit behind them for readers
// that acquire it.  A scalar item needs no scatter: its element is stored here, then published.
__global__ void __launch_bounds__(256)
put_publish_kernel(const DockView dv, const PutBatch batch) {
    uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t it = 0;
    while (it < batch.n_items && i >= batch.item[it].k) { i -= batch.item[it].k; ++it; }
    uint32_t ok = 0, n_oob = 0, n_dup = 0, n_bad = 0, column = 0;
    if (it < batch.n_items) {
        const PutArgs &a = batch.item[it];
        column = a.column;
        const uint32_t L = dv.col_cls[column];
        const uint32_t bit = 1u << column;
        if (L != TD_SCALAR) {
            int32_t s; int64_t l; long long off;
            if (put_entry_live(dv, a, i, L, bit, s, l, off)) {
                __threadfence();
                const uint32_t old = atomicOr(&dv.status[s], bit);
                ok = (old & bit) ? 0u : 1u;
            }
        } else {
            const uint32_t esz = dv.col_esz[column];
            const int32_t s = a.idx[i];
            if (s < 0 || (uint32_t)s >= dv.n) ++n_oob;
            else if ((uint64_t)i >= a.data_elems) ++n_bad;
            else if (dv.status[s] & bit) ++n_dup;
            else {
                if (esz == 4)
                    reinterpret_cast<uint32_t *>(dv.colbase[column])[s] = reinterpret_cast<const uint32_t *>(a.data)[i];
                else
                    reinterpret_cast<uint16_t *>(dv.colbase[column])[s] = reinterpret_cast<const uint16_t *>(a.data)[i];
                __threadfence();
                const uint32_t old = atomicOr(&dv.status[s], bit);
                if (old & bit) ++n_dup; else ok = 1;
            }
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
